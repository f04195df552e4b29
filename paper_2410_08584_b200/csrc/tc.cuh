// Tensor-core (tcgen05 / TMEM) kernels: probe scoring and sparse prefill.
#pragma once
#include "common.cuh"

namespace zipvl {

bool score_tc_supported(const LayerArgs &a, int dtype, int n_probe);
size_t score_tc_ws_bytes(int L, int Hq, int Hkv, int n_probe, int n_seq = 1);
zipvl_status launch_score_tc(const LayerArgs &a, const void *q, const void *k,
                             const int32_t *probe_pos, int P, float *acc, float *norm,
                             double *total, void *ws, int32_t *status_word, cudaStream_t st);

bool prefill_tc_supported(const LayerArgs &a, int dtype);
size_t prefill_tc_ws_bytes(int L, int Hq, int Hkv, int D);
zipvl_status launch_prefill_tc(const LayerArgs &a, const void *q, const void *k, const void *v,
                               const int32_t *idx, const int32_t *k_dev, int k_max, void *out,
                               int out_mode, void *k_cache, void *v_cache, int capacity,
                               int32_t *len_out, void *ws, int32_t *status_word, cudaStream_t st);
// (k_cache == nullptr: attention only; otherwise the kernel also writes K[T], V[T] and *len_out)
// The same call on the kernel with one 128-row query tile per CTA and two CTAs per SM
// (prefill_tc1.cu); launch_prefill_tc picks it for short and medium kept sets.
zipvl_status launch_prefill_tc1(const LayerArgs &a, const void *q, const void *k, const void *v,
                                const int32_t *idx, const int32_t *k_dev, int k_max, void *out,
                                int out_mode, void *k_cache, void *v_cache, int capacity,
                                int32_t *len_out, int32_t *status_word, cudaStream_t st);

}  // namespace zipvl
