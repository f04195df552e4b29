// C ABI of the ZipVL library: argument validation, workspace sizing, dispatch.
// No kernel lives here.  Every entry point validates on the host, launches on
// the caller's stream and returns without synchronising.
#include <math.h>
#include <mutex>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include "common.cuh"
#include "tc.cuh"

namespace zipvl {

static thread_local char g_err[512] = "";

zipvl_status fail(zipvl_status s, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}

zipvl_status check_launch(const char *what) {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "%s: launch failed: %s", what, cudaGetErrorString(e));
    return ZIPVL_OK;
}

static unsigned long long g_launches = 0;
void count_launches(int n) { __atomic_fetch_add(&g_launches, (unsigned long long)n, __ATOMIC_RELAXED); }

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static zipvl_status check_layer(const char *who, const zipvl_layer *l, LayerArgs *a) {
    if (!l) return fail(ZIPVL_ERR_INVALID_ARG, "%s: layer is NULL", who);
    if (l->L < 1) return fail(ZIPVL_ERR_INVALID_ARG, "%s: L = %d < 1", who, l->L);
    if (l->n_q_heads < 1 || l->n_kv_heads < 1 || l->n_q_heads % l->n_kv_heads)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: heads %d / %d", who, l->n_q_heads, l->n_kv_heads);
    if (l->dtype != ZIPVL_BF16 && l->dtype != ZIPVL_F32 && l->dtype != ZIPVL_F16)
        return fail(ZIPVL_ERR_UNSUPPORTED, "%s: dtype %d", who, l->dtype);
    if (l->head_dim != 64 && l->head_dim != 96 && l->head_dim != 128)
        return fail(ZIPVL_ERR_UNSUPPORTED, "%s: head_dim %d (64, 96 or 128)", who, l->head_dim);
    const long long qs = l->q_stride_tok ? l->q_stride_tok : (long long)l->n_q_heads * l->head_dim;
    const long long ks = l->kv_stride_tok ? l->kv_stride_tok : (long long)l->n_kv_heads * l->head_dim;
    if (qs < (long long)l->n_q_heads * l->head_dim || ks < (long long)l->n_kv_heads * l->head_dim ||
        qs % 8 || ks % 8)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: token strides %lld / %lld", who, qs, ks);
    if (!(l->softmax_scale >= 0.f) || isinf(l->softmax_scale))
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: softmax_scale", who);
    a->L = l->L; a->Hq = l->n_q_heads; a->Hkv = l->n_kv_heads; a->D = l->head_dim;
    a->G = l->n_q_heads / l->n_kv_heads;
    a->q_stride = qs; a->kv_stride = ks;
    const float scale = l->softmax_scale > 0.f ? l->softmax_scale : 1.0f / sqrtf((float)l->head_dim);
    a->scale_log2 = scale * kLog2e;
    a->half = (l->dtype == ZIPVL_F16);
    a->n_seq = 1; a->q_seq = 0; a->kv_seq = 0;
    return ZIPVL_OK;
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace zipvl

using namespace zipvl;

extern "C" {

const char *zipvl_status_string(zipvl_status s) {
    switch (s) {
        case ZIPVL_OK: return "ok";
        case ZIPVL_ERR_INVALID_ARG: return "invalid argument";
        case ZIPVL_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case ZIPVL_ERR_WORKSPACE: return "workspace too small";
        case ZIPVL_ERR_CUDA: return "CUDA error";
        case ZIPVL_ERR_TIMEOUT: return "device wait timed out";
        case ZIPVL_ERR_BAD_INDEX: return "index out of range";
    }
    return "unknown status";
}

const char *zipvl_last_error(void) { return g_err; }
int32_t zipvl_version(void) { return 100; }
uint64_t zipvl_launch_count(void) { return __atomic_load_n(&g_launches, __ATOMIC_RELAXED); }

size_t zipvl_workspace_bytes(int32_t op, const zipvl_layer *layer, int32_t n_probe, int32_t batch) {
    LayerArgs a{};
    if (check_layer("workspace_bytes", layer, &a) != ZIPVL_OK) return 0;
    switch (op) {
        case ZIPVL_OP_SCORE:
            if (n_probe < 1) return 0;
            return align256(score_simt_ws_bytes(a.L, a.Hq, n_probe)) +
                   align256(score_tc_ws_bytes(a.L, a.Hq, a.Hkv, n_probe));
        case ZIPVL_OP_SELECT: return select_ws_bytes();
        case ZIPVL_OP_SPARSE_PREFILL: return align256(prefill_tc_ws_bytes(a.L, a.Hq, a.Hkv, a.D)) + 256;
        case ZIPVL_OP_COMPACT_KV: return 256;
        case ZIPVL_OP_DECODE:
            if (batch < 1) return 0;
            return align256(decode_ws_bytes(batch, a.Hq, a.D, a.L, a.Hkv, layer->dtype));
    }
    return 0;
}

zipvl_status zipvl_score(const zipvl_layer *layer, const void *q, const void *k,
                         const int32_t *probe_pos, int32_t n_probe, float *acc, float *norm,
                         double *total, void *ws, size_t ws_bytes, int32_t *status_word,
                         void *stream) {
    LayerArgs a{};
    zipvl_status s = check_layer("zipvl_score", layer, &a);
    if (s != ZIPVL_OK) return s;
    if (!q || !k || !probe_pos || !acc || !norm || !ws)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_score: NULL pointer");
    if (n_probe < 1) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_score: n_probe = %d", n_probe);
    if (!aligned16(q) || !aligned16(k) || !aligned16(ws))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_score: q, k, ws must be 16-byte aligned");
    if (ws_bytes < zipvl_workspace_bytes(ZIPVL_OP_SCORE, layer, n_probe, 1))
        return fail(ZIPVL_ERR_WORKSPACE, "zipvl_score: workspace %zu < %zu", ws_bytes,
                    zipvl_workspace_bytes(ZIPVL_OP_SCORE, layer, n_probe, 1));
    cudaStream_t st = (cudaStream_t)stream;
    if (score_tc_supported(a, layer->dtype, n_probe))
        return launch_score_tc(a, q, k, probe_pos, n_probe, acc, norm, total, ws, status_word, st);
    return launch_score_simt(a, layer->dtype, q, k, probe_pos, n_probe, acc, norm, total, ws,
                             status_word, st);
}

zipvl_status zipvl_select(int32_t L, const float *acc, const float *norm, float tau,
                          uint32_t mode, int32_t fixed_k, int32_t *k_out, int32_t *idx,
                          float *kept_mass, void *ws, size_t ws_bytes, int32_t *status_word,
                          void *stream) {
    if (L < 1 || L > kMaxSelectL) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select: L = %d", L);
    if (!acc || !norm || !k_out || !idx) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select: NULL pointer");
    if (!(tau > 0.f && tau <= 1.f)) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select: tau = %g not in (0,1]", (double)tau);
    if (fixed_k < 0) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select: fixed_k = %d", fixed_k);
    if (mode & 0xFFu & ~(ZIPVL_BUDGET_BY_NORM | ZIPVL_TOPK_BY_ACC))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select: mode = %u", mode);
    if (!ws || ws_bytes < select_ws_bytes())
        return fail(ZIPVL_ERR_WORKSPACE, "zipvl_select: workspace %zu < %zu", ws_bytes, select_ws_bytes());
    if (!aligned16(ws)) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select: ws must be 16-byte aligned");
    return launch_select(L, acc, norm, tau, mode, fixed_k, k_out, idx, kept_mass, ws, status_word,
                         (cudaStream_t)stream);
}

zipvl_status zipvl_sparse_prefill(const zipvl_layer *layer, const void *q, const void *k,
                                  const void *v, const int32_t *idx, const int32_t *k_dev,
                                  int32_t k_max, void *out, int32_t out_mode, void *ws,
                                  size_t ws_bytes, int32_t *status_word, void *stream) {
    LayerArgs a{};
    zipvl_status s = check_layer("zipvl_sparse_prefill", layer, &a);
    if (s != ZIPVL_OK) return s;
    if (!q || !k || !v || !idx || !k_dev || !out)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill: NULL pointer");
    if (k_max < 1 || k_max > a.L)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill: k_max = %d not in [1, L]", k_max);
    if (out_mode != ZIPVL_OUT_PADDED && out_mode != ZIPVL_OUT_COMPACT)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill: out_mode = %d", out_mode);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill: tensors must be 16-byte aligned");
    cudaStream_t st = (cudaStream_t)stream;
    if (prefill_tc_supported(a, layer->dtype)) {
        if (!ws || ws_bytes < zipvl_workspace_bytes(ZIPVL_OP_SPARSE_PREFILL, layer, 0, 1))
            return fail(ZIPVL_ERR_WORKSPACE, "zipvl_sparse_prefill: workspace %zu < %zu", ws_bytes,
                        zipvl_workspace_bytes(ZIPVL_OP_SPARSE_PREFILL, layer, 0, 1));
        return launch_prefill_tc(a, q, k, v, idx, k_dev, k_max, out, out_mode, nullptr, nullptr, 0, nullptr,
                                 ws, status_word, st);
    }
    return launch_prefill_simt(a, layer->dtype, q, k, v, idx, k_dev, k_max, out, out_mode,
                               status_word, st);
}

zipvl_status zipvl_sparse_prefill_compact(const zipvl_layer *layer, const void *q, const void *k,
                                          const void *v, const int32_t *idx, const int32_t *k_dev,
                                          int32_t k_max, void *out, int32_t out_mode, void *k_cache,
                                          void *v_cache, int32_t capacity, int32_t *len_out, void *ws,
                                          size_t ws_bytes, int32_t *status_word, void *stream) {
    LayerArgs a{};
    zipvl_status s = check_layer("zipvl_sparse_prefill_compact", layer, &a);
    if (s != ZIPVL_OK) return s;
    if (!q || !k || !v || !idx || !k_dev || !out || !k_cache || !v_cache || !len_out)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill_compact: NULL pointer");
    if (k_max < 1 || k_max > a.L)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill_compact: k_max = %d not in [1, L]", k_max);
    if (capacity < 1)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill_compact: capacity = %d", capacity);
    if (out_mode != ZIPVL_OUT_PADDED && out_mode != ZIPVL_OUT_COMPACT)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill_compact: out_mode = %d", out_mode);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(k_cache) ||
        !aligned16(v_cache))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_sparse_prefill_compact: tensors must be 16-byte aligned");
    cudaStream_t st = (cudaStream_t)stream;
    if (prefill_tc_supported(a, layer->dtype) && a.kv_stride % 8 == 0) {
        // one kernel: the attention CTAs' spare warps copy the kept K and V rows
        if (!ws || ws_bytes < zipvl_workspace_bytes(ZIPVL_OP_SPARSE_PREFILL, layer, 0, 1))
            return fail(ZIPVL_ERR_WORKSPACE, "zipvl_sparse_prefill_compact: workspace %zu < %zu", ws_bytes,
                        zipvl_workspace_bytes(ZIPVL_OP_SPARSE_PREFILL, layer, 0, 1));
        return launch_prefill_tc(a, q, k, v, idx, k_dev, k_max, out, out_mode, k_cache, v_cache, capacity,
                                 len_out, ws, status_word, st);
    }
    // other shapes and types: the two kernels one after the other
    s = launch_prefill_simt(a, layer->dtype, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
    if (s != ZIPVL_OK) return s;
    return launch_compact(a, elem_bytes(layer->dtype), k, v, idx, k_dev, k_max, k_cache,
                          v_cache, capacity, len_out, status_word, st);
}

zipvl_status zipvl_compact_kv(const zipvl_layer *layer, const void *k, const void *v,
                              const int32_t *idx, const int32_t *k_dev, int32_t k_max,
                              void *k_cache, void *v_cache, int32_t capacity, int32_t *len_out,
                              int32_t *status_word, void *stream) {
    LayerArgs a{};
    zipvl_status s = check_layer("zipvl_compact_kv", layer, &a);
    if (s != ZIPVL_OK) return s;
    if (!k || !v || !idx || !k_dev || !k_cache || !v_cache || !len_out)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_compact_kv: NULL pointer");
    if (k_max < 1 || k_max > a.L)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_compact_kv: k_max = %d not in [1, L]", k_max);
    if (capacity < 1) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_compact_kv: capacity = %d", capacity);
    if (!aligned16(k) || !aligned16(v) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_compact_kv: tensors must be 16-byte aligned");
    return launch_compact(a, elem_bytes(layer->dtype), k, v, idx, k_dev, k_max, k_cache,
                          v_cache, capacity, len_out, status_word, (cudaStream_t)stream);
}

zipvl_status zipvl_decode(const zipvl_decode_desc *d, const void *q, const void *k_new,
                          const void *v_new, void *k_cache, void *v_cache,
                          const int64_t *cache_off, const int32_t *capacity, int32_t *seq_lens,
                          int32_t max_len, void *out, void *ws, size_t ws_bytes,
                          int32_t *status_word, void *stream) {
    if (!d) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_decode: desc is NULL");
    if (d->batch < 1 || d->n_q_heads < 1 || d->n_kv_heads < 1 || d->n_q_heads % d->n_kv_heads)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_decode: batch %d heads %d / %d", d->batch,
                    d->n_q_heads, d->n_kv_heads);
    if (d->batch > 65535) return fail(ZIPVL_ERR_UNSUPPORTED, "zipvl_decode: batch %d > 65535", d->batch);
    if (d->dtype != ZIPVL_BF16 && d->dtype != ZIPVL_F32 && d->dtype != ZIPVL_F16)
        return fail(ZIPVL_ERR_UNSUPPORTED, "zipvl_decode: dtype %d", d->dtype);
    if (d->head_dim != 64 && d->head_dim != 96 && d->head_dim != 128)
        return fail(ZIPVL_ERR_UNSUPPORTED, "zipvl_decode: head_dim %d (64, 96 or 128)", d->head_dim);
    if (d->n_q_heads / d->n_kv_heads > 8 && !decode_tc_supported(*d))
        return fail(ZIPVL_ERR_UNSUPPORTED, "zipvl_decode: more than 8 query heads per kv head (up to 32 "
                                           "in 16-bit storage)");
    if (!q || !k_cache || !v_cache || !cache_off || !capacity || !seq_lens || !out || !ws)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_decode: NULL pointer");
    if ((k_new == NULL) != (v_new == NULL))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_decode: k_new and v_new must both be given or both NULL");
    if (max_len < 1) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_decode: max_len = %d", max_len);
    if (!(d->softmax_scale >= 0.f) || isinf(d->softmax_scale))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_decode: softmax_scale");
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out) || !aligned16(ws))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_decode: tensors must be 16-byte aligned");
    const size_t need = align256(decode_ws_bytes(d->batch, d->n_q_heads, d->head_dim, max_len, d->n_kv_heads, d->dtype));
    if (ws_bytes < need) return fail(ZIPVL_ERR_WORKSPACE, "zipvl_decode: workspace %zu < %zu", ws_bytes, need);
    const float scale = d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / sqrtf((float)d->head_dim);
    return launch_decode(*d, scale * kLog2e, q, k_new, v_new, k_cache, v_cache, cache_off, capacity,
                         seq_lens, max_len, out, ws, status_word, (cudaStream_t)stream);
}

// ---- several sequences of one shape per call -------------------------------------------
static zipvl_status check_batch(const char *who, const zipvl_batch *b, const LayerArgs &a, long long *q_seq,
                                long long *kv_seq) {
    if (!b) return fail(ZIPVL_ERR_INVALID_ARG, "%s: batch is NULL", who);
    if (b->n_seq < 1 || b->n_seq > 4096) return fail(ZIPVL_ERR_INVALID_ARG, "%s: n_seq = %d", who, b->n_seq);
    *q_seq = b->q_stride_seq ? b->q_stride_seq : (long long)a.L * a.q_stride;
    *kv_seq = b->kv_stride_seq ? b->kv_stride_seq : (long long)a.L * a.kv_stride;
    if (*q_seq < (long long)a.L * a.q_stride || *kv_seq < (long long)a.L * a.kv_stride || *q_seq % 8 || *kv_seq % 8)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: sequence strides %lld / %lld", who, *q_seq, *kv_seq);
    return ZIPVL_OK;
}

size_t zipvl_workspace_bytes_batch(int32_t op, const zipvl_layer *layer, int32_t n_probe, int32_t n_seq) {
    LayerArgs a{};
    if (n_seq < 1 || check_layer("workspace_bytes_batch", layer, &a) != ZIPVL_OK) return 0;
    if (op == ZIPVL_OP_SCORE) {
        if (n_probe < 1) return 0;
        return align256(score_simt_ws_bytes(a.L, a.Hq, n_probe)) +
               align256(score_tc_ws_bytes(a.L, a.Hq, a.Hkv, n_probe, n_seq));
    }
    return zipvl_workspace_bytes(op, layer, n_probe, 1);
}

zipvl_status zipvl_score_batch(const zipvl_layer *layer, const zipvl_batch *batch, const void *q,
                               const void *k, const int32_t *probe_pos, int32_t n_probe, float *acc,
                               float *norm, double *total, void *ws, size_t ws_bytes,
                               int32_t *status_word, void *stream) {
    LayerArgs a{};
    zipvl_status s = check_layer("zipvl_score_batch", layer, &a);
    if (s != ZIPVL_OK) return s;
    long long q_seq = 0, kv_seq = 0;
    s = check_batch("zipvl_score_batch", batch, a, &q_seq, &kv_seq);
    if (s != ZIPVL_OK) return s;
    if (!q || !k || !probe_pos || !acc || !norm || !ws)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_score_batch: NULL pointer");
    if (n_probe < 1) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_score_batch: n_probe = %d", n_probe);
    if (!aligned16(q) || !aligned16(k) || !aligned16(ws))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_score_batch: q, k, ws must be 16-byte aligned");
    const size_t need = zipvl_workspace_bytes_batch(ZIPVL_OP_SCORE, layer, n_probe, batch->n_seq);
    if (ws_bytes < need) return fail(ZIPVL_ERR_WORKSPACE, "zipvl_score_batch: workspace %zu < %zu", ws_bytes, need);
    // one launch pair for the whole batch when the tensor-core kernels apply and K is stacked
    // without gaps (one tensor map of n_seq * L rows); otherwise sequence by sequence
    if (score_tc_supported(a, layer->dtype, n_probe) && kv_seq == (long long)a.L * a.kv_stride) {
        a.n_seq = batch->n_seq; a.q_seq = q_seq; a.kv_seq = kv_seq;
        return launch_score_tc(a, q, k, probe_pos, n_probe, acc, norm, total, ws, status_word,
                               (cudaStream_t)stream);
    }
    const size_t eb = elem_bytes(layer->dtype);
    for (int z = 0; z < batch->n_seq; ++z) {
        s = zipvl_score(layer, (const char *)q + (size_t)z * q_seq * eb, (const char *)k + (size_t)z * kv_seq * eb,
                        probe_pos + (size_t)z * n_probe, n_probe, acc + (size_t)z * a.L, norm + (size_t)z * a.L,
                        total ? total + z : nullptr, ws, ws_bytes, status_word, stream);
        if (s != ZIPVL_OK) return s;
    }
    return ZIPVL_OK;
}

zipvl_status zipvl_select_batch(int32_t L, int32_t n_seq, const float *acc, const float *norm, float tau,
                                uint32_t mode, int32_t fixed_k, int32_t *k_out, int32_t *idx,
                                float *kept_mass, void *ws, size_t ws_bytes, int32_t *status_word,
                                void *stream) {
    if (n_seq < 1 || n_seq > 4096) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select_batch: n_seq = %d", n_seq);
    if (L < 1 || L > kMaxSelectL) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select_batch: L = %d", L);
    if (!acc || !norm || !k_out || !idx) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select_batch: NULL pointer");
    if (!(tau > 0.f && tau <= 1.f)) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select_batch: tau = %g not in (0,1]", (double)tau);
    if (fixed_k < 0) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select_batch: fixed_k = %d", fixed_k);
    if (mode & 0xFFu & ~(ZIPVL_BUDGET_BY_NORM | ZIPVL_TOPK_BY_ACC))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select_batch: mode = %u", mode);
    if (!ws || ws_bytes < select_ws_bytes())
        return fail(ZIPVL_ERR_WORKSPACE, "zipvl_select_batch: workspace %zu < %zu", ws_bytes, select_ws_bytes());
    if (!aligned16(ws)) return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_select_batch: ws must be 16-byte aligned");
    return launch_select(L, acc, norm, tau, mode, fixed_k, k_out, idx, kept_mass, ws, status_word,
                         (cudaStream_t)stream, n_seq);
}

zipvl_status zipvl_sparse_prefill_batch(const zipvl_layer *layer, const zipvl_batch *batch, const void *q,
                                        const void *k, const void *v, const int32_t *idx,
                                        const int32_t *k_dev, int32_t k_max, void *out, int32_t out_mode,
                                        void *k_cache, void *v_cache, int32_t capacity, int32_t *len_out,
                                        void *ws, size_t ws_bytes, int32_t *status_word, void *stream) {
    const char *who = "zipvl_sparse_prefill_batch";
    LayerArgs a{};
    zipvl_status s = check_layer(who, layer, &a);
    if (s != ZIPVL_OK) return s;
    long long q_seq = 0, kv_seq = 0;
    s = check_batch(who, batch, a, &q_seq, &kv_seq);
    if (s != ZIPVL_OK) return s;
    if (!q || !k || !v || !idx || !k_dev || !out) return fail(ZIPVL_ERR_INVALID_ARG, "%s: NULL pointer", who);
    const bool caches = (k_cache != nullptr);
    if (caches && (!v_cache || !len_out || capacity < 1))
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: k_cache needs v_cache, len_out and capacity >= 1", who);
    if (k_max < 1 || k_max > a.L) return fail(ZIPVL_ERR_INVALID_ARG, "%s: k_max = %d not in [1, L]", who, k_max);
    if (out_mode != ZIPVL_OUT_PADDED && out_mode != ZIPVL_OUT_COMPACT)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: out_mode = %d", who, out_mode);
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) ||
        (caches && (!aligned16(k_cache) || !aligned16(v_cache))))
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: tensors must be 16-byte aligned", who);
    if (prefill_tc_supported(a, layer->dtype) && a.kv_stride % 8 == 0) {
        if (!ws || ws_bytes < zipvl_workspace_bytes(ZIPVL_OP_SPARSE_PREFILL, layer, 0, 1))
            return fail(ZIPVL_ERR_WORKSPACE, "%s: workspace %zu < %zu", who, ws_bytes,
                        zipvl_workspace_bytes(ZIPVL_OP_SPARSE_PREFILL, layer, 0, 1));
        a.n_seq = batch->n_seq; a.q_seq = q_seq; a.kv_seq = kv_seq;
        return launch_prefill_tc(a, q, k, v, idx, k_dev, k_max, out, out_mode, k_cache, v_cache, capacity,
                                 len_out, ws, status_word, (cudaStream_t)stream);
    }
    // other shapes and types: sequence by sequence through the single-sequence calls
    const size_t eb = elem_bytes(layer->dtype);
    const size_t out_seq = (size_t)(out_mode == ZIPVL_OUT_PADDED ? a.L : k_max) * a.Hq * a.D * eb;
    const size_t cache_seq = (size_t)capacity * a.Hkv * a.D * eb;
    for (int z = 0; z < batch->n_seq; ++z) {
        const char *qz = (const char *)q + (size_t)z * q_seq * eb;
        const char *kz = (const char *)k + (size_t)z * kv_seq * eb, *vz = (const char *)v + (size_t)z * kv_seq * eb;
        if (caches)
            s = zipvl_sparse_prefill_compact(layer, qz, kz, vz, idx + (size_t)z * a.L, k_dev + z, k_max,
                                             (char *)out + z * out_seq, out_mode, (char *)k_cache + z * cache_seq,
                                             (char *)v_cache + z * cache_seq, capacity, len_out + z, ws, ws_bytes,
                                             status_word, stream);
        else
            s = zipvl_sparse_prefill(layer, qz, kz, vz, idx + (size_t)z * a.L, k_dev + z, k_max,
                                     (char *)out + z * out_seq, out_mode, ws, ws_bytes, status_word, stream);
        if (s != ZIPVL_OK) return s;
    }
    return ZIPVL_OK;
}

#define ZIPVL_CUDA(call)                                                                   \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            st_ = fail(ZIPVL_ERR_CUDA, "prefill_layer_host: %s: %s", #call, cudaGetErrorString(e_)); \
            goto done;                                                                     \
        }                                                                                  \
    } while (0)

namespace {
// Device scratch of zipvl_prefill_layer_host comes from a memory pool of the library's own
// (one per device, created on first use) whose release threshold is unlimited: the
// few hundred MB a call needs are then handed back to the pool, not to the driver, when
// the call ends, and the next call gets them again at once.  With the device's default
// pool every call paid for mapping and unmapping that memory (16 ms against 2.7 ms per
// call on a 2944-token layer).  zipvl_release_host_scratch() gives the memory back.
constexpr int kMaxDevices = 64;
cudaMemPool_t g_host_pool[kMaxDevices] = {};
std::mutex g_host_pool_mutex;   // two first calls on one device must not both create a pool

cudaError_t host_pool(cudaMemPool_t *pool) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_host_pool_mutex);
    if (!g_host_pool[dev]) {
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaMemPool_t p = nullptr;
        e = cudaMemPoolCreate(&p, &props);
        if (e != cudaSuccess) return e;
        unsigned long long keep = ~0ull;
        e = cudaMemPoolSetAttribute(p, cudaMemPoolAttrReleaseThreshold, &keep);
        if (e != cudaSuccess) { cudaMemPoolDestroy(p); return e; }
        g_host_pool[dev] = p;
    }
    *pool = g_host_pool[dev];
    return cudaSuccess;
}
}  // namespace

zipvl_status zipvl_release_host_scratch(void) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return fail(ZIPVL_ERR_CUDA, "zipvl_release_host_scratch: no current device");
    std::lock_guard<std::mutex> lock(g_host_pool_mutex);
    if (g_host_pool[dev]) {
        const cudaError_t e = cudaMemPoolTrimTo(g_host_pool[dev], 0);
        if (e != cudaSuccess)
            return fail(ZIPVL_ERR_CUDA, "zipvl_release_host_scratch: %s", cudaGetErrorString(e));
    }
    return ZIPVL_OK;
}

zipvl_status zipvl_prefill_layer_host(const zipvl_layer *layer, const void *q, const void *k,
                                      const void *v, const int32_t *probe_pos, int32_t n_probe,
                                      float tau, int32_t *k_out, int32_t *idx_out, void *out,
                                      void *k_cache_out, void *v_cache_out) {
    return zipvl_layer_step_host(layer, q, k, v, probe_pos, n_probe, tau, k_out, idx_out, out,
                                 k_cache_out, v_cache_out, nullptr, nullptr, nullptr, nullptr);
}

zipvl_status zipvl_layer_step_host(const zipvl_layer *layer, const void *q, const void *k,
                                   const void *v, const int32_t *probe_pos, int32_t n_probe,
                                   float tau, int32_t *k_out, int32_t *idx_out, void *out,
                                   void *k_cache_out, void *v_cache_out, const void *q_new,
                                   const void *k_new, const void *v_new, void *decode_out) {
    LayerArgs a{};
    zipvl_status st_ = check_layer("zipvl_layer_step_host", layer, &a);
    if (st_ != ZIPVL_OK) return st_;
    if (!q || !k || !v || !probe_pos || n_probe < 1)
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_layer_step_host: NULL input or n_probe < 1");
    if (layer->q_stride_tok || layer->kv_stride_tok)
        return fail(ZIPVL_ERR_UNSUPPORTED, "zipvl_layer_step_host: contiguous tensors only");
    const bool with_decode = (q_new != nullptr);
    if (with_decode && (!k_new || !v_new || !decode_out))
        return fail(ZIPVL_ERR_INVALID_ARG, "zipvl_layer_step_host: the decode step needs q_new, k_new, v_new and decode_out");
    if (with_decode && a.G > 8)
        return fail(ZIPVL_ERR_UNSUPPORTED, "zipvl_layer_step_host: more than 8 query heads per kv head");
    const size_t eb = elem_bytes(layer->dtype);
    const size_t qb = (size_t)a.L * a.Hq * a.D * eb, kb = (size_t)a.L * a.Hkv * a.D * eb;
    const size_t ws_score = zipvl_workspace_bytes(ZIPVL_OP_SCORE, layer, n_probe, 1);
    const size_t ws_pf = zipvl_workspace_bytes(ZIPVL_OP_SPARSE_PREFILL, layer, 0, 1);
    size_t ws_b = ws_score > ws_pf ? ws_score : ws_pf;
    if (ws_b < select_ws_bytes()) ws_b = select_ws_bytes();
    // the decode step runs on the cache this call has just compacted: capacity L + 1 rows
    const size_t ws_dec = with_decode ? align256(decode_ws_bytes(1, a.Hq, a.D, a.L + 1, a.Hkv, layer->dtype)) : 0;
    if (ws_b < ws_dec) ws_b = ws_dec;
    const size_t qn_b = (size_t)a.Hq * a.D * eb, kn_b = (size_t)a.Hkv * a.D * eb;
    // one stream-ordered allocation carved into pieces
    size_t off = 0;
    auto carve = [&](size_t bytes) { size_t o = off; off += align256(bytes); return o; };
    const size_t o_q = carve(qb), o_k = carve(kb), o_v = carve(kb), o_out = carve(qb),
                 o_kc = carve(kb + kn_b), o_vc = carve(kb + kn_b), o_probe = carve((size_t)n_probe * 4),
                 o_qn = carve(qn_b), o_kn = carve(kn_b), o_vn = carve(kn_b), o_dec = carve(qn_b),
                 o_acc = carve((size_t)a.L * 4), o_norm = carve((size_t)a.L * 4),
                 o_idx = carve((size_t)a.L * 4), o_misc = carve(256), o_ws = carve(ws_b);
    char *base = nullptr;
    cudaStream_t s = nullptr;
    cudaMemPool_t pool = nullptr;
    int32_t misc[4] = {0, 0, 0, 0};   // k, cache length, device status word, (cache capacity)
    ZIPVL_CUDA(cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking));
    ZIPVL_CUDA(host_pool(&pool));
    ZIPVL_CUDA(cudaMallocFromPoolAsync((void **)&base, off, pool, s));
    {
        int32_t *d_misc = (int32_t *)(base + o_misc);  // [0] k, [1] len, [2] status
        ZIPVL_CUDA(cudaMemsetAsync(d_misc, 0, 256, s));
        ZIPVL_CUDA(cudaMemcpyAsync(base + o_q, q, qb, cudaMemcpyHostToDevice, s));
        ZIPVL_CUDA(cudaMemcpyAsync(base + o_k, k, kb, cudaMemcpyHostToDevice, s));
        ZIPVL_CUDA(cudaMemcpyAsync(base + o_v, v, kb, cudaMemcpyHostToDevice, s));
        ZIPVL_CUDA(cudaMemcpyAsync(base + o_probe, probe_pos, (size_t)n_probe * 4, cudaMemcpyHostToDevice, s));
        if (with_decode) {
            ZIPVL_CUDA(cudaMemcpyAsync(base + o_qn, q_new, qn_b, cudaMemcpyHostToDevice, s));
            ZIPVL_CUDA(cudaMemcpyAsync(base + o_kn, k_new, kn_b, cudaMemcpyHostToDevice, s));
            ZIPVL_CUDA(cudaMemcpyAsync(base + o_vn, v_new, kn_b, cudaMemcpyHostToDevice, s));
        }
        st_ = zipvl_score(layer, base + o_q, base + o_k, (int32_t *)(base + o_probe), n_probe,
                          (float *)(base + o_acc), (float *)(base + o_norm), nullptr, base + o_ws,
                          ws_b, d_misc + 2, s);
        if (st_ != ZIPVL_OK) goto done;
        st_ = zipvl_select(a.L, (float *)(base + o_acc), (float *)(base + o_norm), tau, 0, 0, d_misc,
                           (int32_t *)(base + o_idx), nullptr, base + o_ws, ws_b, d_misc + 2, s);
        if (st_ != ZIPVL_OK) goto done;
        st_ = zipvl_sparse_prefill_compact(layer, base + o_q, base + o_k, base + o_v,
                                           (int32_t *)(base + o_idx), d_misc, a.L, base + o_out,
                                           ZIPVL_OUT_PADDED, base + o_kc, base + o_vc, a.L, d_misc + 1,
                                           base + o_ws, ws_b, d_misc + 2, s);
        if (st_ != ZIPVL_OK) goto done;
        if (with_decode) {
            // Algorithm 2 on the cache just built: d_misc[1] holds its length, d_misc[3] its
            // capacity, d_misc + 4 (8-byte aligned) the one request's offset 0
            const int32_t cap = a.L + 1;
            ZIPVL_CUDA(cudaMemcpyAsync(d_misc + 3, &cap, 4, cudaMemcpyHostToDevice, s));
            zipvl_decode_desc dd = {1, a.Hq, a.Hkv, a.D, layer->dtype, layer->softmax_scale};
            st_ = zipvl_decode(&dd, base + o_qn, base + o_kn, base + o_vn, base + o_kc, base + o_vc,
                               (const int64_t *)(d_misc + 4), d_misc + 3, d_misc + 1, cap, base + o_dec,
                               base + o_ws, ws_b, d_misc + 2, s);
            if (st_ != ZIPVL_OK) goto done;
            ZIPVL_CUDA(cudaMemcpyAsync(decode_out, base + o_dec, qn_b, cudaMemcpyDeviceToHost, s));
        }
        ZIPVL_CUDA(cudaMemcpyAsync(misc, d_misc, sizeof(misc), cudaMemcpyDeviceToHost, s));
        if (out) ZIPVL_CUDA(cudaMemcpyAsync(out, base + o_out, qb, cudaMemcpyDeviceToHost, s));
        if (idx_out) ZIPVL_CUDA(cudaMemcpyAsync(idx_out, base + o_idx, (size_t)a.L * 4, cudaMemcpyDeviceToHost, s));
        ZIPVL_CUDA(cudaStreamSynchronize(s));
        const size_t kept = (size_t)misc[0] * a.Hkv * a.D * eb;
        if (k_cache_out) ZIPVL_CUDA(cudaMemcpyAsync(k_cache_out, base + o_kc, kept, cudaMemcpyDeviceToHost, s));
        if (v_cache_out) ZIPVL_CUDA(cudaMemcpyAsync(v_cache_out, base + o_vc, kept, cudaMemcpyDeviceToHost, s));
        ZIPVL_CUDA(cudaStreamSynchronize(s));
        if (k_out) *k_out = misc[0];
        if (misc[2] != 0)
            st_ = fail(misc[2] & ZIPVL_DEV_TIMEOUT ? ZIPVL_ERR_TIMEOUT : ZIPVL_ERR_BAD_INDEX,
                       "prefill_layer_host: device status word = %d", misc[2]);
    }
done:
    if (base) cudaFreeAsync(base, s);
    if (s) { cudaStreamSynchronize(s); cudaStreamDestroy(s); }
    return st_;
}

}  // extern "C"
