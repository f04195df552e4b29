// KV-cache compaction (Algorithm 1: K = K[T], V = V[T]) -- a pure HBM stream.
//
// Each kept token contributes one contiguous row of Hkv*d elements per tensor.
// The copy is issued as 16-byte chunks, four independent chunks per thread in
// flight, rows walked by a grid sized to fill every SM several times over.
// k is read on the device, so no host synchronisation separates selection
// from compaction.
#include "common.cuh"

namespace zipvl {
namespace {

constexpr int kCpThreads = 256;
constexpr int kCpUnroll = 4;

__global__ void __launch_bounds__(kCpThreads)
compact_kernel(const uint4 *__restrict__ k, const uint4 *__restrict__ v,
               const int32_t *__restrict__ idx, const int32_t *__restrict__ k_dev, int k_max,
               int L, int row_chunks, long long src_row_chunks, uint4 *__restrict__ kc,
               uint4 *__restrict__ vc, int capacity, int32_t *__restrict__ len_out,
               int32_t *status_word) {
    grid_launch_dependents();
    grid_dependency_wait(k, v, idx, k_dev);   // k_dev and idx are the previous kernel's output
    int n = *k_dev;
    const int lim = min(k_max, capacity);
    if (n > lim || n < 0) {
        if (blockIdx.x == 0 && threadIdx.x == 0) report(status_word, ZIPVL_DEV_CAPACITY);
        n = n < 0 ? 0 : lim;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) *len_out = n;

    // chunk counts stay below 2^31 (the launcher checks), so 32-bit division is enough
    const unsigned int total = (unsigned int)n * (unsigned int)row_chunks;   // chunks per tensor
    const unsigned int stride = gridDim.x * kCpThreads;
    const unsigned int rc = (unsigned int)row_chunks;
    for (unsigned int e = blockIdx.x * kCpThreads + threadIdx.x; e < total; e += stride * kCpUnroll) {
        uint4 a[kCpUnroll], b[kCpUnroll];
        long long dst[kCpUnroll];
#pragma unroll
        for (int u = 0; u < kCpUnroll; ++u) {
            const unsigned int ee = e + u * stride;
            dst[u] = -1;
            if (ee < total && ee >= e) {              // (ee >= e: no wrap-around)
                const int i = (int)(ee / rc), c = (int)(ee % rc);
                const int t = idx[i];
                if (t < 0 || t >= L) {
                    report(status_word, ZIPVL_DEV_BAD_INDEX);
                } else {
                    const long long src = (long long)t * src_row_chunks + c;
                    a[u] = __ldg(k + src);
                    b[u] = __ldg(v + src);
                    dst[u] = ee;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kCpUnroll; ++u) {
            if (dst[u] >= 0) {
                kc[dst[u]] = a[u];
                vc[dst[u]] = b[u];
            }
        }
    }
}

}  // namespace

zipvl_status launch_compact(const LayerArgs &a, int elem_bytes, const void *k, const void *v,
                            const int32_t *idx, const int32_t *k_dev, int k_max, void *k_cache,
                            void *v_cache, int capacity, int32_t *len_out, int32_t *status_word,
                            cudaStream_t st) {
    const long long row_bytes = (long long)a.Hkv * a.D * elem_bytes;
    const long long src_row_bytes = a.kv_stride * elem_bytes;
    if (row_bytes % 16 || src_row_bytes % 16)
        return fail(ZIPVL_ERR_INVALID_ARG, "compact_kv: rows must be multiples of 16 bytes");
    const int row_chunks = (int)(row_bytes / 16);
    const long long total = (long long)k_max * row_chunks;
    long long blocks = (total + (long long)kCpThreads * kCpUnroll - 1) / (kCpThreads * kCpUnroll);
    if ((long long)k_max * row_chunks >= (1LL << 31) || (long long)capacity * row_chunks >= (1LL << 31))
        return fail(ZIPVL_ERR_INVALID_ARG, "compact_kv: more than 2^31 16-byte chunks per tensor");
    const long long cap = 148LL * 8;      // one resident wave: 8 CTAs of 256 threads per SM
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const cudaError_t e = launch_dependent(compact_kernel, dim3((unsigned)blocks), dim3(kCpThreads), 0, st,
                                           (const uint4 *)k, (const uint4 *)v, idx, k_dev, k_max, a.L,
                                           row_chunks, src_row_bytes / 16, (uint4 *)k_cache,
                                           (uint4 *)v_cache, capacity, len_out, status_word);
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "compact_kv: launch: %s", cudaGetErrorString(e));
    count_launches(1);
    return check_launch("zipvl_compact_kv");
}

}  // namespace zipvl
