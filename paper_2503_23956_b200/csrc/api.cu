// Exported C ABI: host-side argument checks, workspace carve-up and dispatch to the kernel launchers.
// Every check happens before anything is enqueued, so a failing call leaves the stream untouched.
#include <math.h>
#include <string.h>

#include <vector>

#include "common.cuh"
#include "ptx.cuh"

namespace aircache {

static thread_local int g_last_cuda_error = 0;

void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

int check_shape(const aircache_shape_t *s) {
    if (!s) return AIRCACHE_ERR_INVALID_ARG;
    if (s->n_layers < 1 || s->batch < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->head_dim < 1 ||
        s->n_visual < 1 || s->n_text < 1 || s->window < 1 || s->slack < 0)
        return AIRCACHE_ERR_INVALID_ARG;
    if (!(s->scale > 0.0f) || !isfinite(s->scale)) return AIRCACHE_ERR_INVALID_ARG;
    if (s->window > s->n_text) return AIRCACHE_ERR_INVALID_ARG;
    if (s->n_q_heads % s->n_kv_heads != 0) return AIRCACHE_ERR_INVALID_ARG;
    if (s->head_dim != 64 && s->head_dim != 128) return AIRCACHE_ERR_UNSUPPORTED;
    if (s->n_kv_heads != 1 && s->n_kv_heads != 2 && s->n_kv_heads != 4 && s->n_kv_heads != 8)
        return AIRCACHE_ERR_UNSUPPORTED;
    if (s->n_q_heads / s->n_kv_heads > kMaxGroup) return AIRCACHE_ERR_UNSUPPORTED;
    if (s->window > kMaxWindow) return AIRCACHE_ERR_UNSUPPORTED;
    if (s->n_visual < 3) return AIRCACHE_ERR_UNSUPPORTED;
    if (s->per_kv_head != 0 && s->per_kv_head != 1) return AIRCACHE_ERR_INVALID_ARG;
    if (n_cells(s) > kMaxRegions) return AIRCACHE_ERR_UNSUPPORTED;
    if ((int64_t)s->n_visual + s->n_text + s->slack > (1 << 24)) return AIRCACHE_ERR_UNSUPPORTED;
    return AIRCACHE_OK;
}

int check_full(const aircache_shape_t *s, const aircache_full_t *f) {
    if (!f || !f->k || !f->v) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)f->k & 15) || ((uintptr_t)f->v & 15)) return AIRCACHE_ERR_ALIGNMENT;
    const int64_t st[4] = {f->stride_layer, f->stride_batch, f->stride_head, f->stride_token};
    for (int i = 0; i < 4; ++i) {
        if (st[i] < 0) return AIRCACHE_ERR_INVALID_ARG;
        if (st[i] % 8 != 0) return AIRCACHE_ERR_ALIGNMENT;
    }
    if (f->stride_token < s->head_dim && s->n_visual + s->n_text > 1) return AIRCACHE_ERR_INVALID_ARG;
    return AIRCACHE_OK;
}

int64_t kept_per_sequence(const aircache_shape_t *s, double ratio) {
    int64_t cells = (int64_t)s->n_visual * (int64_t)s->n_layers * cells_of(s);
    return (int64_t)floor(ratio * (double)cells + 0.5);
}

WsLayout ws_layout(const aircache_shape_t *s) {
    WsLayout w;
    const int64_t LB = (int64_t)s->n_layers * s->batch;
    const int64_t groups = LB * s->n_kv_heads;
    const int64_t cap = score_row_cap(s);
    int64_t off = 0;
    auto take = [&](int64_t bytes) {
        int64_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    w.status = take(256);
    w.tickets = take((int64_t)kMaxRegions * 4);
    w.plan_memo = take(kPlanMemoBytes);
    w.row_count = take(groups * 4);
    w.row_info = take(groups * cap * 4);
    w.row_coef = take(groups * cap * 4);
    w.row_text = take(groups * cap * 8);
    w.chunk_stats = take(score_chunk_cells(s) * cap * 8);
    w.row_final = take(groups * cap * 8);
    w.group_ticket = take(groups * 4);
    w.dispatch = take(256);
    w.imp_part = take(s->per_kv_head ? 256 : groups * (int64_t)s->n_visual * 4);
    w.q_block = take(groups * 16 * (int64_t)s->head_dim * 2);
    w.mom_strength = take(n_cells(s) * 8);
    w.mom_skew = take(n_cells(s) * 8);
    w.kept = take(n_cells(s) * s->n_visual * 4);
    w.partials = take((int64_t)2 * kMaxDecodeCtas * partial_slot_floats(s->n_q_heads, s->head_dim) * 4);
    w.total = off;
    return w;
}

static int check_ws(const aircache_shape_t *s, void *ws, int64_t bytes) {
    if (!ws) return AIRCACHE_ERR_INVALID_ARG;
    if ((uintptr_t)ws & 255) return AIRCACHE_ERR_ALIGNMENT;
    if (bytes < ws_layout(s).total) return AIRCACHE_ERR_WORKSPACE_TOO_SMALL;
    return AIRCACHE_OK;
}

static int check_ragged(const aircache_shape_t *s, const aircache_ragged_t *c, bool need_kv) {
    if (!c || !c->offsets || !c->lens) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)c->offsets & 7) || ((uintptr_t)c->lens & 3)) return AIRCACHE_ERR_ALIGNMENT;
    if (c->first_row < 0) return AIRCACHE_ERR_INVALID_ARG;
    if (need_kv) {
        if (!c->k || !c->v) return AIRCACHE_ERR_INVALID_ARG;
        if (((uintptr_t)c->k & 127) || ((uintptr_t)c->v & 127)) return AIRCACHE_ERR_ALIGNMENT;
        if (c->total_rows < 1 || c->total_rows >= ((int64_t)1 << 31)) return AIRCACHE_ERR_CAPACITY;
        if (c->first_row >= c->total_rows) return AIRCACHE_ERR_CAPACITY;
    }
    (void)s;
    return AIRCACHE_OK;
}

// ---------------------------------------------------------------------------------------------
// aircache_selftest_wait_timeout: the bounded wait on a barrier that nobody completes
// ---------------------------------------------------------------------------------------------
namespace {
__global__ void wait_timeout_kernel(uint32_t *status) {
    __shared__ uint64_t s_bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&s_bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s_abort = 0;
    }
    __syncthreads();
    // no thread ever arrives: every waiter gives up after kSpinLimit polls (or as soon as one of them has),
    // the first one records the status word
    mbar_wait(smem_u32(&s_bar), 0, &s_abort, status, 9);
}
}  // namespace

int launch_selftest_timeout(void *ws, cudaStream_t st) {
    wait_timeout_kernel<<<1, 64, 0, st>>>(reinterpret_cast<uint32_t *>(ws));
    AIRCACHE_LAUNCH_CHECK();
    return AIRCACHE_OK;
}

}  // namespace aircache

using namespace aircache;

extern "C" {

int aircache_version(void) { return AIRCACHE_VERSION; }

const char *aircache_strerror(int code) {
    switch (code) {
        case AIRCACHE_OK: return "success";
        case AIRCACHE_ERR_INVALID_ARG: return "invalid argument";
        case AIRCACHE_ERR_UNSUPPORTED: return "shape not supported by the sm_100a kernels";
        case AIRCACHE_ERR_ALIGNMENT: return "pointer or stride breaks the alignment rules";
        case AIRCACHE_ERR_WORKSPACE_TOO_SMALL: return "workspace smaller than aircache_workspace_bytes()";
        case AIRCACHE_ERR_CAPACITY: return "ragged cache capacity too small";
        case AIRCACHE_ERR_CUDA: return "CUDA error (see aircache_last_cuda_error)";
        case AIRCACHE_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case AIRCACHE_ERR_STATIC_SCRATCH:
            return "problem needs more scratch than the built-in array of aircache_decode_attn_static holds";
        case AIRCACHE_ERR_INCONSISTENT:
            return "budgets, offsets or kept lists on the device do not fit the buffers; the rows concerned were not written";
        default: return "unknown error code";
    }
}

int aircache_last_cuda_error(void) { return g_last_cuda_error; }

int64_t aircache_kept_per_sequence(const aircache_shape_t *shape, double ratio) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!(ratio >= 0.0 && ratio <= 1.0)) return AIRCACHE_ERR_INVALID_ARG;
    return kept_per_sequence(shape, ratio);
}

int64_t aircache_total_rows(const aircache_shape_t *shape, double ratio) {
    int64_t t = aircache_kept_per_sequence(shape, ratio);
    if (t < 0) return t;
    return (int64_t)shape->batch * (t + (int64_t)shape->n_layers * cells_of(shape) * ((int64_t)shape->n_text + shape->slack));
}

int64_t aircache_workspace_bytes(const aircache_shape_t *shape) {
    int rc = check_shape(shape);
    if (rc) return rc;
    return ws_layout(shape).total;
}

int aircache_score_layers(const aircache_shape_t *shape, const aircache_full_t *full, const void *q_window,
                          float alpha, int32_t layer_begin, int32_t layer_count, float *scores,
                          uint64_t *elite_mask, void *workspace, int64_t workspace_bytes, void *cuda_stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if ((rc = check_full(shape, full))) return rc;
    if (!q_window || !scores) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)q_window & 15) || ((uintptr_t)scores & 15) || ((uintptr_t)elite_mask & 7))
        return AIRCACHE_ERR_ALIGNMENT;
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return AIRCACHE_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_count < 0 || layer_begin > shape->n_layers - layer_count)
        return AIRCACHE_ERR_INVALID_ARG;
    if ((rc = check_ws(shape, workspace, workspace_bytes))) return rc;
    if (layer_count == 0) return AIRCACHE_OK;
    return launch_score(shape, full, q_window, alpha, layer_begin, layer_count, scores, elite_mask, workspace,
                        (cudaStream_t)cuda_stream);
}

int aircache_score(const aircache_shape_t *shape, const aircache_full_t *full, const void *q_window, float alpha,
                   float *scores, uint64_t *elite_mask, void *workspace, int64_t workspace_bytes,
                   void *cuda_stream) {
    if (!shape) return AIRCACHE_ERR_INVALID_ARG;
    return aircache_score_layers(shape, full, q_window, alpha, 0, shape->n_layers, scores, elite_mask, workspace,
                                 workspace_bytes, cuda_stream);
}

int aircache_budget(const aircache_shape_t *shape, const float *scores, double ratio, int32_t mode,
                    int32_t *budgets, double *strength, double *skewness, aircache_ragged_t *layout,
                    void *workspace, int64_t workspace_bytes, void *cuda_stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!scores || !budgets) return AIRCACHE_ERR_INVALID_ARG;
    if (!(ratio >= 0.0 && ratio <= 1.0) || mode < 0 || mode > 3) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)scores & 3) || ((uintptr_t)budgets & 3) || ((uintptr_t)strength & 7) ||
        ((uintptr_t)skewness & 7))
        return AIRCACHE_ERR_ALIGNMENT;
    if ((rc = check_ragged(shape, layout, false))) return rc;
    if ((rc = check_ws(shape, workspace, workspace_bytes))) return rc;
    return launch_budget(shape, scores, ratio, mode, budgets, strength, skewness, layout, workspace,
                         (cudaStream_t)cuda_stream);
}

int aircache_compact(const aircache_shape_t *shape, const aircache_full_t *full, const float *scores,
                     const int32_t *budgets, double ratio, aircache_ragged_t *out, int32_t *kept_idx,
                     void *workspace, int64_t workspace_bytes, void *cuda_stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if ((rc = check_full(shape, full))) return rc;
    if (!scores || !budgets) return AIRCACHE_ERR_INVALID_ARG;
    if (!(ratio >= 0.0 && ratio <= 1.0)) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)scores & 3) || ((uintptr_t)budgets & 3) || ((uintptr_t)kept_idx & 3))
        return AIRCACHE_ERR_ALIGNMENT;
    if ((rc = check_ragged(shape, out, true))) return rc;
    if (out->total_rows < out->first_row + aircache_total_rows(shape, ratio)) return AIRCACHE_ERR_CAPACITY;
    if ((rc = check_ws(shape, workspace, workspace_bytes))) return rc;
    return launch_compact(shape, full, scores, budgets, ratio, out, kept_idx, workspace,
                          (cudaStream_t)cuda_stream);
}

int aircache_decode_attn(const aircache_shape_t *shape, const aircache_ragged_t *cache, const void *q, float *out,
                         void *workspace, int64_t workspace_bytes, void *cuda_stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if ((rc = check_ragged(shape, cache, true))) return rc;
    if (!q || !out) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return AIRCACHE_ERR_ALIGNMENT;
    if ((rc = check_ws(shape, workspace, workspace_bytes))) return rc;
    return launch_decode(shape, cache, q, nullptr, nullptr, out, workspace, (cudaStream_t)cuda_stream);
}

int aircache_decode_step(const aircache_shape_t *shape, aircache_ragged_t *cache, const void *q, const void *k_new,
                         const void *v_new, int32_t appended, float *out, void *workspace, int64_t workspace_bytes,
                         void *cuda_stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if ((rc = check_ragged(shape, cache, true))) return rc;
    if (!q || !out || !k_new || !v_new || appended < 0) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15) || ((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15))
        return AIRCACHE_ERR_ALIGNMENT;
    if (appended >= shape->slack) return AIRCACHE_ERR_CAPACITY;
    if ((rc = check_ws(shape, workspace, workspace_bytes))) return rc;
    return launch_decode(shape, cache, q, k_new, v_new, out, workspace, (cudaStream_t)cuda_stream);
}

int aircache_decode_attn_static(const aircache_shape_t *shape, const aircache_ragged_t *cache, const void *q,
                                float *out, void *cuda_stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if ((rc = check_ragged(shape, cache, true))) return rc;
    if (!q || !out) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15) || ((uintptr_t)out & 15)) return AIRCACHE_ERR_ALIGNMENT;
    return launch_decode_static(shape, cache, q, out, (cudaStream_t)cuda_stream);
}

int aircache_append(const aircache_shape_t *shape, aircache_ragged_t *cache, const void *k_new, const void *v_new,
                    int32_t appended, void *cuda_stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if ((rc = check_ragged(shape, cache, true))) return rc;
    if (!k_new || !v_new || appended < 0) return AIRCACHE_ERR_INVALID_ARG;
    if (((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15)) return AIRCACHE_ERR_ALIGNMENT;
    if (appended >= shape->slack) return AIRCACHE_ERR_CAPACITY;
    return launch_append(shape, cache, k_new, v_new, appended, (cudaStream_t)cuda_stream);
}

int aircache_reset_status(void *workspace, int64_t workspace_bytes, void *cuda_stream) {
    if (!workspace) return AIRCACHE_ERR_INVALID_ARG;
    if ((uintptr_t)workspace & 255) return AIRCACHE_ERR_ALIGNMENT;
    if (workspace_bytes < kResetBytes) return AIRCACHE_ERR_WORKSPACE_TOO_SMALL;
    AIRCACHE_CUDA_TRY(cudaMemsetAsync(workspace, 0, kResetBytes, (cudaStream_t)cuda_stream));
    return AIRCACHE_OK;
}

int aircache_check_status(void *workspace, int64_t workspace_bytes, void *cuda_stream) {
    if (!workspace) return AIRCACHE_ERR_INVALID_ARG;
    if ((uintptr_t)workspace & 255) return AIRCACHE_ERR_ALIGNMENT;
    if (workspace_bytes < 256) return AIRCACHE_ERR_WORKSPACE_TOO_SMALL;
    uint32_t word = 0;
    AIRCACHE_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost,
                                      (cudaStream_t)cuda_stream));
    AIRCACHE_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    if (word == kStatusInconsistent) return AIRCACHE_ERR_INCONSISTENT;
    return word ? AIRCACHE_ERR_TIMEOUT : AIRCACHE_OK;
}

int aircache_selftest_wait_timeout(void *workspace, int64_t workspace_bytes, void *cuda_stream) {
    if (!workspace) return AIRCACHE_ERR_INVALID_ARG;
    if ((uintptr_t)workspace & 255) return AIRCACHE_ERR_ALIGNMENT;
    if (workspace_bytes < kStatusBytes) return AIRCACHE_ERR_WORKSPACE_TOO_SMALL;
    return launch_selftest_timeout(workspace, (cudaStream_t)cuda_stream);
}

// Device address of a host range if all of it is page-locked memory the GPU can read in place, else null.
static void *mapped_host_range(const void *p, int64_t bytes) {
    if (!p || bytes < 1) return nullptr;
    void *first = nullptr, *last = nullptr;
    const char *c = static_cast<const char *>(p);
    if (cudaHostGetDevicePointer(&first, const_cast<char *>(c), 0) != cudaSuccess ||
        cudaHostGetDevicePointer(&last, const_cast<char *>(c + bytes - 1), 0) != cudaSuccess) {
        cudaGetLastError();   // pageable memory: not an error of the caller's, and not a sticky one
        return nullptr;
    }
    if (!first || static_cast<char *>(last) - static_cast<char *>(first) != bytes - 1) return nullptr;
    return first;
}

int aircache_host_range_is_mapped(const void *host_ptr, int64_t bytes) {
    return mapped_host_range(host_ptr, bytes) ? 1 : 0;
}

int aircache_pipeline_host(const aircache_shape_t *shape, const aircache_full_t *h_full, int64_t full_elems,
                           void *d_full_k, void *d_full_v, const void *h_q_window, void *d_q_window,
                           const void *h_q_steps, void *d_q_steps, int32_t n_steps, float alpha, double ratio,
                           int32_t mode, float *d_scores, int32_t *d_budgets, aircache_ragged_t *d_cache,
                           float *d_out, float *h_out, int32_t *h_budgets, void *workspace,
                           int64_t workspace_bytes, void *cuda_stream) {
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!h_full || !h_full->k || !h_full->v || !d_full_k || !d_full_v || !h_q_window || !d_q_window ||
        !h_q_steps || !d_q_steps || !d_scores || !d_budgets || !d_cache || !d_out || !h_out || !h_budgets)
        return AIRCACHE_ERR_INVALID_ARG;
    if (full_elems < 1 || n_steps < 0) return AIRCACHE_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int64_t LB = (int64_t)shape->n_layers * shape->batch;
    const int64_t qw_bytes = LB * shape->window * shape->n_q_heads * shape->head_dim * 2;
    const int64_t q_elems = LB * shape->n_q_heads * shape->head_dim;
    aircache_full_t d_full = *h_full;
    d_full.k = d_full_k;
    d_full.v = d_full_v;
    // K is read twice in full by the scoring passes, so it is uploaded.  V is read once, and only the rows that
    // survive (kept visual rows and text rows): when the host buffer is page-locked and mapped, the gather
    // kernel reads those rows from it in place and the upload of the other rows never happens.
    void *v_in_place = mapped_host_range(h_full->v, full_elems * 2);
    if (v_in_place) d_full.v = v_in_place;
    // validate everything the stages will check before the first copy is enqueued
    if ((rc = check_full(shape, &d_full))) return rc;
    if ((rc = check_ragged(shape, d_cache, true))) return rc;
    if (d_cache->total_rows < d_cache->first_row + aircache_total_rows(shape, ratio)) return AIRCACHE_ERR_CAPACITY;
    if ((rc = check_ws(shape, workspace, workspace_bytes))) return rc;
    if (!(alpha >= 0.0f && alpha <= 1.0f) || !(ratio >= 0.0 && ratio <= 1.0) || mode < 0 || mode > 3)
        return AIRCACHE_ERR_INVALID_ARG;

    // From here on work is in flight on the stream (and later on the copy stream) that reads and writes the
    // caller's host buffers: whatever happens, the call returns only after both streams have drained.
    constexpr int32_t kCopyEvery = 16;   // decode rounds per upload of queries
    constexpr int32_t kDownEvery = 4;    // decode rounds per download of outputs (the last block's copy is the tail)
    struct CopySide {
        cudaStream_t main = nullptr, stream = nullptr, up = nullptr;
        cudaEvent_t event = nullptr;
        std::vector<cudaEvent_t> arrived;   // one per block of kCopyEvery rounds: its queries are on the device
        ~CopySide() {
            if (up) cudaStreamSynchronize(up);
            if (stream) cudaStreamSynchronize(stream);
            cudaStreamSynchronize(main);
            if (event) cudaEventDestroy(event);
            for (cudaEvent_t e : arrived) cudaEventDestroy(e);
            if (stream) cudaStreamDestroy(stream);
            if (up) cudaStreamDestroy(up);
        }
    } side;
    side.main = st;
    AIRCACHE_CUDA_TRY(cudaMemcpyAsync(d_full_k, h_full->k, full_elems * 2, cudaMemcpyHostToDevice, st));
    if (!v_in_place)
        AIRCACHE_CUDA_TRY(cudaMemcpyAsync(d_full_v, h_full->v, full_elems * 2, cudaMemcpyHostToDevice, st));
    AIRCACHE_CUDA_TRY(cudaMemcpyAsync(d_q_window, h_q_window, qw_bytes, cudaMemcpyHostToDevice, st));
    // The decode queries are needed round by round only: a third stream uploads them, kCopyEvery rounds at a
    // time, behind the caches (which the compression is waiting for) and beside the compression and the
    // earlier rounds; a round waits for the event of its block.
    if (n_steps > 0) {
        AIRCACHE_CUDA_TRY(cudaStreamCreateWithFlags(&side.stream, cudaStreamNonBlocking));
        AIRCACHE_CUDA_TRY(cudaStreamCreateWithFlags(&side.up, cudaStreamNonBlocking));
        AIRCACHE_CUDA_TRY(cudaEventCreateWithFlags(&side.event, cudaEventDisableTiming));
        AIRCACHE_CUDA_TRY(cudaEventRecord(side.event, st));
        AIRCACHE_CUDA_TRY(cudaStreamWaitEvent(side.up, side.event, 0));
        for (int32_t first = 0; first < n_steps; first += kCopyEvery) {
            const int32_t n = n_steps - first < kCopyEvery ? n_steps - first : kCopyEvery;
            AIRCACHE_CUDA_TRY(cudaMemcpyAsync((char *)d_q_steps + (int64_t)first * q_elems * 2,
                                              (const char *)h_q_steps + (int64_t)first * q_elems * 2,
                                              (int64_t)n * q_elems * 2, cudaMemcpyHostToDevice, side.up));
            cudaEvent_t e = nullptr;
            AIRCACHE_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
            side.arrived.push_back(e);
            AIRCACHE_CUDA_TRY(cudaEventRecord(e, side.up));
        }
    }
    if ((rc = aircache_reset_status(workspace, workspace_bytes, st))) return rc;
    if ((rc = aircache_score(shape, &d_full, d_q_window, alpha, d_scores, nullptr, workspace, workspace_bytes, st)))
        return rc;
    if ((rc = aircache_budget(shape, d_scores, ratio, mode, d_budgets, nullptr, nullptr, d_cache, workspace,
                              workspace_bytes, st)))
        return rc;
    if ((rc = aircache_compact(shape, &d_full, d_scores, d_budgets, ratio, d_cache, nullptr, workspace,
                               workspace_bytes, st)))
        return rc;
    // The results go back to the host while later rounds still run: a second stream copies every
    // kDownEvery rounds' outputs as soon as the round that wrote the last of them has finished.
    for (int32_t i = 0; i < n_steps; ++i) {
        if (i % kCopyEvery == 0) AIRCACHE_CUDA_TRY(cudaStreamWaitEvent(st, side.arrived[i / kCopyEvery], 0));
        const char *q = (const char *)d_q_steps + (int64_t)i * q_elems * 2;
        if ((rc = aircache_decode_attn(shape, d_cache, q, d_out + (int64_t)i * q_elems, workspace,
                                       workspace_bytes, st)))
            return rc;
        if ((i + 1) % kDownEvery == 0 || i + 1 == n_steps) {
            const int32_t first = i / kDownEvery * kDownEvery;
            AIRCACHE_CUDA_TRY(cudaEventRecord(side.event, st));
            AIRCACHE_CUDA_TRY(cudaStreamWaitEvent(side.stream, side.event, 0));
            AIRCACHE_CUDA_TRY(cudaMemcpyAsync(h_out + (int64_t)first * q_elems, d_out + (int64_t)first * q_elems,
                                              (int64_t)(i + 1 - first) * q_elems * 4, cudaMemcpyDeviceToHost,
                                              side.stream));
        }
    }
    AIRCACHE_CUDA_TRY(cudaMemcpyAsync(h_budgets, d_budgets, n_cells(shape) * 4, cudaMemcpyDeviceToHost, st));
    if (n_steps > 0) {
        AIRCACHE_CUDA_TRY(cudaStreamSynchronize(side.up));
        AIRCACHE_CUDA_TRY(cudaStreamSynchronize(side.stream));
    }
    AIRCACHE_CUDA_TRY(cudaStreamSynchronize(st));
    return AIRCACHE_OK;
}

}  // extern "C"
