// Shared device / host helpers of the ZipVL CUDA library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/zipvl.h"

namespace zipvl {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kMaxSelectL = 1 << 20;

// thread-local error text (api.cu)
zipvl_status fail(zipvl_status s, const char *fmt, ...);
zipvl_status check_launch(const char *what);
void count_launches(int n);  // kernels launched by this library so far (zipvl_launch_count)

__device__ __forceinline__ void report(int32_t *status_word, uint32_t bits) {
    if (status_word) atomicOr(reinterpret_cast<unsigned int *>(status_word), bits);
}

// ---- element access: 8 consecutive elements as floats ----------------------
__device__ __forceinline__ void load8(const float *p, float (&x)[8]) {
    const float4 a = *reinterpret_cast<const float4 *>(p);
    const float4 b = *reinterpret_cast<const float4 *>(p + 4);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
    x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void unpack8(const uint4 r, float (&x)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&x)[8]) {
    unpack8(*reinterpret_cast<const uint4 *>(p), x);
}
__device__ __forceinline__ void unpack8h(const uint4 r, float (&x)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
    }
}
__device__ __forceinline__ void load8(const __half *p, float (&x)[8]) {
    unpack8h(*reinterpret_cast<const uint4 *>(p), x);
}
__device__ __forceinline__ float to_float(__half v) { return __half2float(v); }
__device__ __forceinline__ void store_elem(__half *p, float v) { *p = __float2half_rn(v); }
inline int elem_bytes(int dtype) { return dtype == ZIPVL_F32 ? 4 : 2; }
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void store_elem(float *p, float v) { *p = v; }
__device__ __forceinline__ void store_elem(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// order-preserving map float -> uint32 (larger float, larger key)
__device__ __forceinline__ uint32_t float_key(float v) {
    const uint32_t b = __float_as_uint(v);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// ---- programmatic dependent launch ------------------------------------------------
// Every kernel of the hot path is launched with the programmatic-stream-serialization
// attribute and begins with grid_launch_dependents(): the next kernel in the stream
// may then be staged (and run its prologue up to its own grid_dependency_wait()) while
// this one is still running, once all of this one's CTAs have started.  A kernel
// touches global memory only behind grid_dependency_wait(), which returns when every
// earlier kernel in the stream has completed and its writes are visible.  Next to a
// kernel launched without the attribute both instructions do nothing.
//
// The pointers through which the kernel then reads what an earlier kernel wrote are handed
// to the wait and come back "redefined" by an empty asm statement.  Without that, a load
// through a `const T *__restrict__` parameter -- or through any restrict parameter the
// kernel never stores to -- counts as a load of invariant memory, which the compiler may
// schedule above every barrier, the wait included: a decode step replayed from a CUDA
// graph read the cache length of the replay before, because that one load had moved up.
template <typename T>
__device__ __forceinline__ void redefine_pointer(T &p) { asm volatile("" : "+l"(p)::"memory"); }
template <typename... P>
__device__ __forceinline__ void grid_dependency_wait(P &...ptrs) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    (redefine_pointer(ptrs), ...);
}
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                             cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- launchers implemented per file -----------------------------------------
struct LayerArgs {
    int L, Hq, Hkv, D, G;
    long long q_stride, kv_stride;  // elements per token
    float scale_log2;               // softmax scale * log2(e)
    int half;                       // 16-bit storage is IEEE half (1) or bfloat16 (0)
    // a batch of n_seq sequences of this shape (1 for the single-sequence calls): elements
    // between the sequences of Q and of K / V; per-sequence outputs are stacked likewise
    int n_seq;
    long long q_seq, kv_seq;
};

zipvl_status launch_score_simt(const LayerArgs &a, int dtype, const void *q, const void *k,
                               const int32_t *probe_pos, int P, float *acc, float *norm,
                               double *total, void *ws, int32_t *status_word, cudaStream_t st);
size_t score_simt_ws_bytes(int L, int Hq, int P);

zipvl_status launch_select(int L, const float *acc, const float *norm, float tau, uint32_t mode,
                           int fixed_k, int32_t *k_out, int32_t *idx, float *kept_mass, void *ws,
                           int32_t *status_word, cudaStream_t st, int n_seq = 1);
size_t select_ws_bytes();

zipvl_status launch_prefill_simt(const LayerArgs &a, int dtype, const void *q, const void *k,
                                 const void *v, const int32_t *idx, const int32_t *k_dev,
                                 int k_max, void *out, int out_mode, int32_t *status_word,
                                 cudaStream_t st);

zipvl_status launch_compact(const LayerArgs &a, int elem_bytes, const void *k, const void *v,
                            const int32_t *idx, const int32_t *k_dev, int k_max, void *k_cache,
                            void *v_cache, int capacity, int32_t *len_out, int32_t *status_word,
                            cudaStream_t st);

// Paged cache: request b's row r lives in page table[b * stride + (r >> shift)] of a pool of
// n_pages pages of (1 << shift) rows each.  table == nullptr: contiguous caches at cache_off.
struct PageArgs {
    const int32_t *table;
    int stride, shift, n_pages;
};

// (Hkv and dtype decide whether the grouped-query tensor-core kernel, which leaves more partials,
// may run: 0 / -1 = the CUDA-core layout)
size_t decode_ws_bytes(int B, int Hq, int D, int max_len, int Hkv = 0, int dtype = -1);
int decode_chunk_rows(int B, int Hq, int max_len);
size_t decode_partial_bytes(int B, int Hq, int D, int max_len);
// used != nullptr: used[b * (Hq / group) + hq / group] of the n_chunks slots hold a partial
zipvl_status launch_decode_merge(int dtype, int D, int Hq, int B, int chunk, int n_chunks, const float *ws,
                                 const int *lens, int32_t *seq_lens, void *out, cudaStream_t st,
                                 const int *used = nullptr, int group = 1);
// Grouped-query decode on the tensor cores: 16-bit storage, head_dim 64 / 96 / 128, 2 to 32 query
// heads per kv head.  Two kernels that leave partials in the layout of the kernels in decode.cu and the
// (length, appended) pairs in lens[]; the caller launches the merge.
//   decode_tc.cu             one CTA per chunk of a (request, kv head): one partial per chunk, returns
//                            the chunk it used (never smaller than min_chunk);
//   decode_tc_persistent.cu  one CTA per SM over an equal share of all tiles (large batches): four
//                            partials per CTA and (request, kv head), n_slots per (request, query
//                            head), the number in use per (request, kv head) in used[].
bool decode_tc_supported(const zipvl_decode_desc &d);
zipvl_status launch_decode_tc(const zipvl_decode_desc &d, float scale_log2, const void *q,
                              const void *k_new, const void *v_new, void *k_cache, void *v_cache,
                              const int64_t *cache_off, PageArgs pg, const int32_t *capacity,
                              int32_t *seq_lens, int max_len, int min_chunk, float *partials, int *lens,
                              int32_t *status_word, cudaStream_t st, int *chunk_out);
zipvl_status launch_decode_tcp(const zipvl_decode_desc &d, float scale_log2, const void *q,
                               const void *k_new, const void *v_new, void *k_cache, void *v_cache,
                               const int64_t *cache_off, PageArgs pg, const int32_t *capacity,
                               int32_t *seq_lens, int max_len, int n_slots, float *partials, int *lens,
                               int *used, int32_t *status_word, cudaStream_t st);
zipvl_status launch_decode(const zipvl_decode_desc &d, float scale_log2, const void *q,
                           const void *k_new, const void *v_new, void *k_cache, void *v_cache,
                           const int64_t *cache_off, const int32_t *capacity, int32_t *seq_lens,
                           int max_len, void *out, void *ws, int32_t *status_word,
                           cudaStream_t st);

}  // namespace zipvl
