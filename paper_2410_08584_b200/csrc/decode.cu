// Decode attention over the kept cache (Algorithm 2; Eq. 4-5) for a ragged
// batch -- an HBM stream of every cached key and value, read exactly once.
//
// Two kernels per step, the second a small programmatic dependent of the first:
//   grid = (cache chunk, kv head x query-head tile, request).  A row of one kv
//   head (d elements) is read by d*sizeof/16 adjacent lanes with one 16-byte load
//   each; the lanes of a row reduce the dot product by shuffles and keep an
//   online softmax (base 2) for up to 8 query heads that share the kv head, so
//   grouped-query attention still reads each cached byte once.  Four rows per
//   lane group are in flight before any is consumed.
//   Append (Eq. 4): the CTA whose chunk holds row seq_lens[b] takes that row from
//   k_new / v_new and stores it into the cache on the way.
//   Each CTA leaves (m, l, o) for its chunk in the workspace.  The merge kernel
//   (staged while the first one runs, so its launch costs nothing) combines the
//   chunks of every (request, head), writes the output and bumps seq_lens[b]; it
//   reads the step's length from the workspace, where the first kernel left it.
// Lengths live on the device; the host only supplies an upper bound.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace zipvl {
namespace {

constexpr int kDecThreads = 128;

__device__ __forceinline__ uint4 ld_stream(const void *p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

template <typename T> struct Epl;
template <> struct Epl<__nv_bfloat16> { static constexpr int v = 8; };
template <> struct Epl<float> { static constexpr int v = 4; };
template <> struct Epl<__half> { static constexpr int v = 8; };

template <typename T, int N>
__device__ __forceinline__ void unpack(const uint4 r, float (&x)[N]);
template <>
__device__ __forceinline__ void unpack<__nv_bfloat16, 8>(const uint4 r, float (&x)[8]) {
    unpack8(r, x);
}
template <>
__device__ __forceinline__ void unpack<__half, 8>(const uint4 r, float (&x)[8]) {
    unpack8h(r, x);
}
template <>
__device__ __forceinline__ void unpack<float, 4>(const uint4 r, float (&x)[4]) {
    x[0] = __uint_as_float(r.x); x[1] = __uint_as_float(r.y);
    x[2] = __uint_as_float(r.z); x[3] = __uint_as_float(r.w);
}

// kDecUnroll: rows per lane group in flight before any is consumed (8 where the registers allow)
// kPaged: the cache rows are found through a block table (a separate instantiation, so that the
// contiguous path carries none of its address arithmetic)
template <typename T, int D, int GT, int kDecUnroll, bool kPaged>
__global__ void __launch_bounds__(kDecThreads)
decode_kernel(int Hq, int Hkv, float scale_log2, const T *__restrict__ q,
              const T *__restrict__ k_new, const T *__restrict__ v_new, T *__restrict__ k_cache,
              T *__restrict__ v_cache, const int64_t *__restrict__ cache_off, PageArgs pg,
              const int32_t *__restrict__ capacity, int32_t *__restrict__ seq_lens, int max_len,
              int chunk, int n_chunks, float *__restrict__ ws, int *__restrict__ lens,
              T *__restrict__ out, int32_t *status_word) {
    constexpr int EPL = Epl<T>::v;          // elements per lane (16 bytes)
    constexpr int LPR_USED = D / EPL;       // lanes that hold a piece of a row
    // lanes per row: a power of two (the dot product is reduced by xor shuffles); with head_dim
    // 96 the last quarter of them holds nothing
    constexpr int LPR = LPR_USED <= 8 ? 8 : (LPR_USED <= 16 ? 16 : 32);
    constexpr int RPW = 32 / LPR;           // rows per warp per load
    constexpr int NG = (kDecThreads / 32) * RPW;
    __shared__ float sm_o[NG][GT][D];
    __shared__ float sm_m[NG][GT], sm_l[NG][GT];

    grid_launch_dependents();
    // lengths and caches may be the previous kernel's output
    grid_dependency_wait(q, k_new, v_new, k_cache, v_cache, cache_off, capacity, seq_lens, pg.table);
    const int G = Hq / Hkv;
    const int q_tiles = (G + GT - 1) / GT;
    const int hkv = blockIdx.y / q_tiles, qt = blockIdx.y % q_tiles;
    const int b = blockIdx.z;
    const int h0 = hkv * G + qt * GT;        // first query head of this CTA
    const int n_heads = min(GT, G - qt * GT);
    const bool first = blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0;
    // the query rows do not depend on the lengths: their loads go out together with them
    float qv[GT][EPL];
    {
        const int lr_q = (threadIdx.x & 31) % LPR;
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            if (g < n_heads && lr_q < LPR_USED) {
                const uint4 r = *reinterpret_cast<const uint4 *>(
                    q + ((long long)b * Hq + h0 + g) * D + lr_q * EPL);
                unpack<T, EPL>(r, qv[g]);
            } else {
#pragma unroll
                for (int e = 0; e < EPL; ++e) qv[g][e] = 0.f;
            }
        }
    }

    // Eq. 4: the new row goes to position seq_lens[b] if the cache has room
    // A request whose length is negative or beyond its capacity, or whose cache offset breaks
    // the 16-byte alignment of the row loads, is skipped as a whole (no load, no append, a
    // zero output) and reported: none of its rows can be trusted to lie inside the cache.
    const int old_len = seq_lens[b];
    const int cap = capacity[b];
    const long long coff = kPaged ? 0ll : cache_off[b];
    const bool bad = old_len < 0 || old_len > cap || ((coff * (long long)sizeof(T)) & 15) != 0;
    if (bad && first) report(status_word, ZIPVL_DEV_BAD_INDEX);
    const bool appended = !bad && k_new != nullptr && old_len < cap;
    if (k_new != nullptr && !bad && !appended && first) report(status_word, ZIPVL_DEV_CAPACITY);
    int len = bad ? 0 : old_len + (appended ? 1 : 0);
    if (len > max_len) {
        if (first) report(status_word, ZIPVL_DEV_CAPACITY);
        len = max_len;
    }
    const int new_row = appended ? old_len : -1;
    const int c0 = blockIdx.x * chunk;
    const bool valid = c0 < len;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rg = warp * RPW + lane / LPR;  // row group of this lane
    const int lr = lane % LPR;               // lane inside the row
    const bool live = lr < LPR_USED;         // (head_dim 96: 12 of 16 lanes)

    if (valid) {
        const int c1 = min(len, c0 + chunk);
        float o[GT][EPL], m[GT], l[GT];
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            m[g] = -INFINITY;
            l[g] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) { o[g][e] = 0.f; qv[g][e] *= scale_log2; }
        }

        const long long row_pitch = (long long)Hkv * D;
        const long long head_off = (long long)hkv * D + lr * EPL;
        T *kb = k_cache + coff + head_off;
        T *vb = v_cache + coff + head_off;
        // element offset of a cache row from kb / vb; -1 for a page outside the pool (reported,
        // the row is skipped)
        const int32_t *my_table = kPaged ? pg.table + (long long)b * pg.stride : nullptr;
        auto row_off = [&](int row) -> long long {
            if (!kPaged) return row * row_pitch;
            const int page = my_table[row >> pg.shift];
            if (page < 0 || page >= pg.n_pages) { report(status_word, ZIPVL_DEV_BAD_INDEX); return -1; }
            return (((long long)page << pg.shift) + (row & ((1 << pg.shift) - 1))) * row_pitch;
        };

        for (int base = c0; base < c1; base += NG * kDecUnroll) {
            uint4 kk[kDecUnroll], vv[kDecUnroll];
            bool ok[kDecUnroll];
#pragma unroll
            for (int u = 0; u < kDecUnroll; ++u) {
                const int row = base + u * NG + rg;
                ok[u] = row < c1;
                const long long ro = ok[u] ? row_off(row) : -1;
                ok[u] = ok[u] && ro >= 0;
                if (!live) {
                    kk[u] = make_uint4(0, 0, 0, 0);
                    vv[u] = make_uint4(0, 0, 0, 0);
                } else if (ok[u] && row != new_row) {
                    kk[u] = ld_stream(kb + ro);
                    vv[u] = ld_stream(vb + ro);
                } else if (ok[u]) {
                    // the appended token: read it from k_new / v_new, store it on the way
                    kk[u] = *reinterpret_cast<const uint4 *>(k_new + (long long)b * row_pitch + head_off);
                    vv[u] = *reinterpret_cast<const uint4 *>(v_new + (long long)b * row_pitch + head_off);
                    if (qt == 0) {
                        *reinterpret_cast<uint4 *>(kb + ro) = kk[u];
                        *reinterpret_cast<uint4 *>(vb + ro) = vv[u];
                    }
                } else {
                    kk[u] = make_uint4(0, 0, 0, 0);
                    vv[u] = make_uint4(0, 0, 0, 0);
                }
            }
            float s[kDecUnroll][GT];
#pragma unroll
            for (int u = 0; u < kDecUnroll; ++u) {
                float kf[EPL];
                unpack<T, EPL>(kk[u], kf);
#pragma unroll
                for (int g = 0; g < GT; ++g) {
                    float d = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) d = fmaf(qv[g][e], kf[e], d);
#pragma unroll
                    for (int off = LPR / 2; off > 0; off >>= 1)
                        d += __shfl_xor_sync(0xffffffffu, d, off);
                    s[u][g] = ok[u] ? d : -INFINITY;
                }
            }
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                float mn = m[g];
#pragma unroll
                for (int u = 0; u < kDecUnroll; ++u) mn = fmaxf(mn, s[u][g]);
                if (mn == -INFINITY) continue;
                const float sc = fast_exp2(m[g] - mn);
                m[g] = mn;
                l[g] *= sc;
#pragma unroll
                for (int e = 0; e < EPL; ++e) o[g][e] *= sc;
#pragma unroll
                for (int u = 0; u < kDecUnroll; ++u) s[u][g] = fast_exp2(s[u][g] - mn);
            }
#pragma unroll
            for (int u = 0; u < kDecUnroll; ++u) {
                float vf[EPL];
                unpack<T, EPL>(vv[u], vf);
#pragma unroll
                for (int g = 0; g < GT; ++g) {
                    const float p = (m[g] == -INFINITY) ? 0.f : s[u][g];
                    l[g] += p;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) o[g][e] = fmaf(p, vf[e], o[g][e]);
                }
            }
        }

        // combine the row groups of the CTA
#pragma unroll
        for (int g = 0; g < GT; ++g) {
#pragma unroll
            for (int e = 0; e < EPL; ++e)
                if (live) sm_o[rg][g][lr * EPL + e] = o[g][e];
            if (lr == 0) { sm_m[rg][g] = m[g]; sm_l[rg][g] = l[g]; }
        }
        __syncthreads();
        for (int t = threadIdx.x; t < n_heads * D; t += kDecThreads) {
            const int g = t / D, c = t % D;
            float M = -INFINITY;
#pragma unroll
            for (int r = 0; r < NG; ++r) M = fmaxf(M, sm_m[r][g]);
            float Ls = 0.f, Os = 0.f;
#pragma unroll
            for (int r = 0; r < NG; ++r) {
                const float mr = sm_m[r][g];
                const float w = (mr == -INFINITY) ? 0.f : fast_exp2(mr - M);
                Ls += sm_l[r][g] * w;
                Os += sm_o[r][g][c] * w;
            }
            float *dst = ws + (((long long)b * Hq + h0 + g) * n_chunks + blockIdx.x) * (D + 2);
            dst[2 + c] = Os;
            if (c == 0) { dst[0] = M; dst[1] = Ls; }
        }
    } else if ((int)threadIdx.x < n_heads) {
        // a chunk past the request's length: an empty partial (the merge reads every chunk slot
        // without waiting for the length)
        float *dst = ws + (((long long)b * Hq + h0 + threadIdx.x) * n_chunks + blockIdx.x) * (D + 2);
        dst[0] = -INFINITY;
        dst[1] = 0.f;
    }

    // the length this step attends over, for the merge kernel (which must not read
    // seq_lens: it also writes it)
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        lens[2 * b] = len;
        lens[2 * b + 1] = appended ? 1 : 0;
    }
}

// Second kernel of a step: merges the per-chunk partial results of one request's query
// heads (online-softmax merge), writes the output, and bumps the request's length.
// Launched as a programmatic dependent of the kernel above, so it is staged while that one
// runs; no tickets, no counters to clear.  `lanes` (1, 2, 4 or 8) adjacent lanes share two
// channels of one head: lane p takes chunks p, p + lanes, ... -- every chunk slot holds a
// partial, an empty one past the request's length, so all loads go out at once without waiting
// for the length -- and the lanes are merged by shuffles in a fixed order.  The host picks
// `lanes` so that a batch of many requests does not become thousands of CTAs with one load
// each (merge_lanes below).
__device__ __forceinline__ void store2(float *p, float a, float b) { *reinterpret_cast<float2 *>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(__nv_bfloat16 *p, float a, float b) {
    *reinterpret_cast<__nv_bfloat162 *>(p) = __floats2bfloat162_rn(a, b);
}
__device__ __forceinline__ void store2(__half *p, float a, float b) { *reinterpret_cast<__half2 *>(p) = __floats2half2_rn(a, b); }

// kMergeUnroll: slots per lane in flight.  8 behind the CUDA-core kernel; 6 behind the tensor-core
// kernels, which keeps the merge at 48 registers: its CTAs then fit beside a persistent decode CTA
// (544 threads x 96 registers) and wait there, staged, while that kernel runs.
template <typename T, int D, int kMergeUnroll>
__global__ void __launch_bounds__(256, kMergeUnroll == 8 ? 4 : 5)
decode_merge_kernel(int Hq, int lanes, int n_chunks, const float *__restrict__ ws,
                    const int *__restrict__ lens, int32_t *__restrict__ seq_lens, T *__restrict__ out,
                    const int *__restrict__ used, int group) {
    static_assert(D % 2 == 0, "two channels per thread");
    grid_launch_dependents();
    grid_dependency_wait(ws, lens, seq_lens, used);
    const int b = blockIdx.y;
    const int t = (blockIdx.x * 256 + threadIdx.x) / lanes;             // (head, channel pair) of this lane group
    const int part = threadIdx.x % lanes;
    const bool live = t < Hq * (D / 2);
    const int hq = live ? t / (D / 2) : 0, c = live ? 2 * (t % (D / 2)) : 0;
    const float *src = ws + ((long long)b * Hq + hq) * n_chunks * (D + 2);
    // the tensor-core kernel fills only the first used[request, kv head] slots of a head
    const int n_used = used ? min(n_chunks, max(0, used[b * (Hq / group) + hq / group])) : n_chunks;
    float M = -INFINITY, Ls = 0.f, O0 = 0.f, O1 = 0.f;
    for (int i0 = part; i0 < n_used; i0 += kMergeUnroll * lanes) {
        float2 ml[kMergeUnroll], oi[kMergeUnroll];
#pragma unroll
        for (int u = 0; u < kMergeUnroll; ++u) {
            const int i = i0 + u * lanes;
            const bool in = live && i < n_used;
            const float *p = src + (long long)(in ? i : 0) * (D + 2);   // (a slot is (D + 2) * 4 bytes: 8-byte aligned)
            ml[u] = in ? __ldcg(reinterpret_cast<const float2 *>(p)) : make_float2(-INFINITY, 0.f);
            oi[u] = in ? __ldcg(reinterpret_cast<const float2 *>(p + 2 + c)) : make_float2(0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kMergeUnroll; ++u) {
            if (ml[u].x != -INFINITY) {
                const float Mn = fmaxf(M, ml[u].x);
                const float wo = fast_exp2(M - Mn), wn = fast_exp2(ml[u].x - Mn);
                Ls = Ls * wo + ml[u].y * wn;
                O0 = O0 * wo + oi[u].x * wn;
                O1 = O1 * wo + oi[u].y * wn;
                M = Mn;
            }
        }
    }
    for (int o = 1; o < lanes; o <<= 1) {
        const float M2 = __shfl_xor_sync(0xffffffffu, M, o);
        const float L2 = __shfl_xor_sync(0xffffffffu, Ls, o);
        const float P0 = __shfl_xor_sync(0xffffffffu, O0, o);
        const float P1 = __shfl_xor_sync(0xffffffffu, O1, o);
        const float Mn = fmaxf(M, M2);
        // (the two sides of a pair compute the same sum in the same order of operands)
        const float w1 = (M == -INFINITY) ? 0.f : fast_exp2(M - Mn);
        const float w2 = (M2 == -INFINITY) ? 0.f : fast_exp2(M2 - Mn);
        const bool lo = (part & o) == 0;
        Ls = lo ? (Ls * w1 + L2 * w2) : (L2 * w2 + Ls * w1);
        O0 = lo ? (O0 * w1 + P0 * w2) : (P0 * w2 + O0 * w1);
        O1 = lo ? (O1 * w1 + P1 * w2) : (P1 * w2 + O1 * w1);
        M = Mn;
    }
    // (an empty cache with nothing appended has only empty partials: the output is zero)
    if (live && part == 0)
        store2(out + ((long long)b * Hq + hq) * D + c, Ls > 0.f ? O0 / Ls : 0.f, Ls > 0.f ? O1 / Ls : 0.f);
    // Eq. 4: the appended row now counts
    if (blockIdx.x == 0 && threadIdx.x == 0 && lens[2 * b + 1]) seq_lens[b] = lens[2 * b];
}

// Lanes per (head, channel pair) of the merge: as many as there are slots to share (at most
// 8), but no more than keep the whole launch within about one wave of threads -- with hundreds
// of requests the merge is bound by the number of CTAs it starts, not by its loads.
int merge_lanes(int B, int Hq, int D, int n_slots) {
    int lanes = 8;
    while (lanes > 1 && (lanes / 2 >= n_slots || (long long)B * Hq * (D / 2) * lanes > 148LL * 2048)) lanes >>= 1;
    return lanes;
}
dim3 merge_grid(int B, int Hq, int D, int lanes) { return dim3((Hq * (D / 2) * lanes + 255) / 256, B); }

// Cache rows per CTA: small problems get small chunks so that every SM still has
// several CTAs in flight (about eight per SM), large ones stream 512 rows per CTA.
int decode_chunk(int B, int Hq, int max_len) {
    const long long target = (long long)B * Hq * max_len / (148 * 8);
    int c = 32;
    while (c < target && c < 512) c <<= 1;
    return c;
}

// partials per (request, query head) in the workspace: one per chunk for the CUDA-core kernel and
// the chunked tensor-core kernel; the persistent tensor-core kernel cuts the work by tiles (a
// request of c chunks' worth of tiles may be shared by c + 1 CTAs) and leaves four partials per CTA
int partial_slots(int B, int Hq, int max_len, bool tc) {
    const int chunk = decode_chunk(B, Hq, max_len);
    const int n_chunks = (max_len + chunk - 1) / chunk;
    return tc ? 4 * (n_chunks + 1) : n_chunks;
}
bool tc_shape(int Hq, int Hkv, int D, int dtype) {
    if (Hkv < 1 || Hq % Hkv) return false;
    const zipvl_decode_desc d = {1, Hq, Hkv, D, dtype, 0.f};
    return decode_tc_supported(d);
}

size_t partial_bytes(int B, int Hq, int D, int max_len, bool tc = false) {
    if (tc) return ((size_t)B * Hq * partial_slots(B, Hq, max_len, true) * (D + 2) * sizeof(float) + 255) & ~(size_t)255;
    const int chunk = decode_chunk(B, Hq, max_len);
    const size_t n_slots = (max_len + chunk - 1) / chunk;
    return ((size_t)B * Hq * n_slots * (D + 2) * sizeof(float) + 255) & ~(size_t)255;
}
// (length, appended) per request, and for the tensor-core kernel the slots in use per (request, kv head)
size_t counter_bytes(int B, int Hq) { return (size_t)(2 * B + B * Hq) * sizeof(int); }

template <typename T, int D>
zipvl_status run(const zipvl_decode_desc &d, float scale_log2, const void *q, const void *k_new,
                 const void *v_new, void *k_cache, void *v_cache, const int64_t *cache_off, PageArgs pg,
                 const int32_t *capacity, int32_t *seq_lens, int max_len, void *out, void *ws,
                 int32_t *status_word, cudaStream_t st) {
    const int B = d.batch, Hq = d.n_q_heads, Hkv = d.n_kv_heads, G = Hq / Hkv;
    const int chunk = decode_chunk(B, Hq, max_len);
    const int n_chunks = (max_len + chunk - 1) / chunk;
    float *wsf = reinterpret_cast<float *>(ws);
    int *lens = reinterpret_cast<int *>(reinterpret_cast<char *>(ws) + partial_bytes(B, Hq, D, max_len));
#define ZIPVL_DEC_P(GT_, P_)                                                                    \
    {                                                                                           \
        dim3 grid(n_chunks, Hkv * ((G + GT_ - 1) / GT_), B);                                    \
        le = launch_dependent(decode_kernel<T, D, GT_, (GT_ <= 2 ? 8 : 4), P_>, grid, dim3(kDecThreads), 0, st, \
                              Hq, Hkv, scale_log2, (const T *)q, (const T *)k_new, (const T *)v_new,  \
                              (T *)k_cache, (T *)v_cache, cache_off, pg, capacity, seq_lens, max_len, \
                              chunk, n_chunks, wsf, lens, (T *)out, status_word);                    \
    }
#define ZIPVL_DEC(GT_)                                                                          \
    {                                                                                           \
        if (pg.table) ZIPVL_DEC_P(GT_, true)                                                    \
        else ZIPVL_DEC_P(GT_, false)                                                            \
    }
    cudaError_t le = cudaSuccess;
    if (G == 1) ZIPVL_DEC(1)
    else if (G == 2) ZIPVL_DEC(2)
    else if (G <= 4) ZIPVL_DEC(4)
    else ZIPVL_DEC(8)
#undef ZIPVL_DEC
#undef ZIPVL_DEC_P
    if (le == cudaSuccess) {
        const int lanes = merge_lanes(B, Hq, D, n_chunks);
        le = launch_dependent(decode_merge_kernel<T, D, 8>, merge_grid(B, Hq, D, lanes), dim3(256), 0, st, Hq,
                              lanes, n_chunks, (const float *)wsf, (const int *)lens, seq_lens, (T *)out,
                              (const int *)nullptr, 1);
    }
    if (le != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "zipvl_decode: launch: %s", cudaGetErrorString(le));
    count_launches(2);
    return check_launch("zipvl_decode");
}

}  // namespace

// what the decode over a quantised cache (kvquant.cu) shares with this file: the chunking, the
// layout of the partial results and the merge kernel
int decode_chunk_rows(int B, int Hq, int max_len) { return decode_chunk(B, Hq, max_len); }
size_t decode_partial_bytes(int B, int Hq, int D, int max_len) { return partial_bytes(B, Hq, D, max_len); }
zipvl_status launch_decode_merge(int dtype, int D, int Hq, int B, int chunk, int n_chunks, const float *ws,
                                 const int *lens, int32_t *seq_lens, void *out, cudaStream_t st,
                                 const int *used, int group) {
    cudaError_t le = cudaErrorInvalidValue;
    (void)chunk;
    const int lanes = merge_lanes(B, Hq, D, n_chunks);
    const dim3 grid = merge_grid(B, Hq, D, lanes);
#define ZIPVL_MERGE(T_, D_) \
    le = launch_dependent(decode_merge_kernel<T_, D_, 6>, grid, dim3(256), 0, st, Hq, lanes, n_chunks, ws, lens, seq_lens, (T_ *)out, used, group)
    if (dtype == ZIPVL_BF16 && D == 128) ZIPVL_MERGE(__nv_bfloat16, 128);
    else if (dtype == ZIPVL_BF16 && D == 96) ZIPVL_MERGE(__nv_bfloat16, 96);
    else if (dtype == ZIPVL_BF16 && D == 64) ZIPVL_MERGE(__nv_bfloat16, 64);
    else if (dtype == ZIPVL_F16 && D == 128) ZIPVL_MERGE(__half, 128);
    else if (dtype == ZIPVL_F16 && D == 96) ZIPVL_MERGE(__half, 96);
    else if (dtype == ZIPVL_F16 && D == 64) ZIPVL_MERGE(__half, 64);
#undef ZIPVL_MERGE
    if (le != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "decode merge: launch: %s", cudaGetErrorString(le));
    count_launches(1);
    return ZIPVL_OK;
}

size_t decode_ws_bytes(int B, int Hq, int D, int max_len, int Hkv, int dtype) {
    return partial_bytes(B, Hq, D, max_len, tc_shape(Hq, Hkv, D, dtype)) + counter_bytes(B, Hq);
}

namespace {
zipvl_status dispatch_decode(const zipvl_decode_desc &d, float scale_log2, const void *q,
                             const void *k_new, const void *v_new, void *k_cache, void *v_cache,
                             const int64_t *cache_off, PageArgs pg, const int32_t *capacity,
                             int32_t *seq_lens, int max_len, void *out, void *ws,
                             int32_t *status_word, cudaStream_t st) {
    // Grouped-query attention in 16-bit storage runs on the tensor cores from two query heads per
    // kv head on: there the CUDA-core kernel is bound by its multiply-adds (0.49 of the HBM copy
    // rate at four heads per kv head, 0.29 at seven; at two it reaches 0.81 against 0.84).  Of the
    // two tensor-core kernels the persistent one takes the large problems (from about ten
    // key/value tiles per SM on it is 5 to 15 % faster: no CTA prologue between work items); below
    // that the launch of one CTA per chunk is quicker (fewer partials to merge, shorter CTAs).
    // ZIPVL_DECODE_KERNEL=simt|tc|tcp overrides the choice (measurements, tests).
    {
        const char *env = getenv("ZIPVL_DECODE_KERNEL");
        const int G = d.n_q_heads / d.n_kv_heads;
        const long long tiles = (long long)d.batch * d.n_kv_heads * ((max_len + 127) / 128);
        constexpr long long kPersistentFrom = 1500;
        const bool want_simt = env && !strcmp(env, "simt");
        if (decode_tc_supported(d) && (!want_simt || G > 8)) {
            const int B = d.batch, Hq = d.n_q_heads, D = d.head_dim;
            const bool persistent = env && !strcmp(env, "tcp") ? true
                                    : (env && !strcmp(env, "tc") ? false : tiles >= kPersistentFrom);
            float *wsf = reinterpret_cast<float *>(ws);
            int *lens = reinterpret_cast<int *>(reinterpret_cast<char *>(ws) + partial_bytes(B, Hq, D, max_len, true));
            int *used = lens + 2 * B;
            int chunk = decode_chunk(B, Hq, max_len);
            zipvl_status sm;
            if (persistent) {
                const int n_slots = partial_slots(B, Hq, max_len, true);    // as the workspace was sized
                const zipvl_status s = launch_decode_tcp(d, scale_log2, q, k_new, v_new, k_cache, v_cache,
                                                         cache_off, pg, capacity, seq_lens, max_len, n_slots, wsf,
                                                         lens, used, status_word, st);
                if (s != ZIPVL_OK) return s;
                sm = launch_decode_merge(d.dtype, D, Hq, B, chunk, n_slots, wsf, lens, seq_lens, out, st, used, G);
            } else {
                const zipvl_status s = launch_decode_tc(d, scale_log2, q, k_new, v_new, k_cache, v_cache, cache_off,
                                                        pg, capacity, seq_lens, max_len, chunk, wsf, lens,
                                                        status_word, st, &chunk);
                if (s != ZIPVL_OK) return s;
                sm = launch_decode_merge(d.dtype, D, Hq, B, chunk, (max_len + chunk - 1) / chunk, wsf, lens,
                                         seq_lens, out, st);
            }
            return sm != ZIPVL_OK ? sm : check_launch("zipvl_decode");
        }
        if (G > 8) return fail(ZIPVL_ERR_UNSUPPORTED, "decode: %d query heads per kv head", G);
    }
#define ZIPVL_ARGS d, scale_log2, q, k_new, v_new, k_cache, v_cache, cache_off, pg, capacity, \
                   seq_lens, max_len, out, ws, status_word, st
    if (d.dtype == ZIPVL_BF16) {
        if (d.head_dim == 128) return run<__nv_bfloat16, 128>(ZIPVL_ARGS);
        if (d.head_dim == 96) return run<__nv_bfloat16, 96>(ZIPVL_ARGS);
        if (d.head_dim == 64) return run<__nv_bfloat16, 64>(ZIPVL_ARGS);
    } else if (d.dtype == ZIPVL_F16) {
        if (d.head_dim == 128) return run<__half, 128>(ZIPVL_ARGS);
        if (d.head_dim == 96) return run<__half, 96>(ZIPVL_ARGS);
        if (d.head_dim == 64) return run<__half, 64>(ZIPVL_ARGS);
    } else {
        if (d.head_dim == 128) return run<float, 128>(ZIPVL_ARGS);
        if (d.head_dim == 96) return run<float, 96>(ZIPVL_ARGS);
        if (d.head_dim == 64) return run<float, 64>(ZIPVL_ARGS);
    }
#undef ZIPVL_ARGS
    return fail(ZIPVL_ERR_UNSUPPORTED, "decode: head_dim %d", d.head_dim);
}
}  // namespace

zipvl_status launch_decode(const zipvl_decode_desc &d, float scale_log2, const void *q,
                           const void *k_new, const void *v_new, void *k_cache, void *v_cache,
                           const int64_t *cache_off, const int32_t *capacity, int32_t *seq_lens,
                           int max_len, void *out, void *ws, int32_t *status_word,
                           cudaStream_t st) {
    return dispatch_decode(d, scale_log2, q, k_new, v_new, k_cache, v_cache, cache_off,
                           PageArgs{nullptr, 0, 0, 0}, capacity, seq_lens, max_len, out, ws, status_word, st);
}

// ---- decode without any allocation ------------------------------------------
// Scratch for zipvl_decode_noalloc: the per-chunk (m, l, o) partials and the
// per-request (length, appended) pairs live in this file-scope device array
// instead of a caller-supplied workspace.  Every GPU that loads the library holds these 8 MiB until the
// process exits.
constexpr size_t kNoAllocScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_decode_scratch[kNoAllocScratchBytes];

// The array's name is only a host-side stand-in in host code, so the device
// address is looked up once per device (with that device current) and cached.
constexpr int kMaxDevices = 64;
static void *g_scratch_addr[kMaxDevices];   // zero-initialised: "not looked up yet"

static zipvl_status noalloc_scratch(void **ptr) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess)
        return fail(ZIPVL_ERR_CUDA, "zipvl_decode_noalloc: cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(ZIPVL_ERR_UNSUPPORTED, "zipvl_decode_noalloc: device ordinal %d", dev);
    void *p = __atomic_load_n(&g_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        e = cudaGetSymbolAddress(&p, g_decode_scratch);
        if (e != cudaSuccess || !p)
            return fail(ZIPVL_ERR_CUDA, "zipvl_decode_noalloc: cudaGetSymbolAddress: %s",
                        cudaGetErrorString(e));
        __atomic_store_n(&g_scratch_addr[dev], p, __ATOMIC_RELEASE);
    }
    *ptr = p;
    return ZIPVL_OK;
}

}  // namespace zipvl

extern "C" zipvl_status zipvl_decode_noalloc(const zipvl_decode_desc *d, const void *q,
                                             const void *k_new, const void *v_new, void *k_cache,
                                             void *v_cache, const int64_t *cache_off,
                                             const int32_t *capacity, int32_t *seq_lens,
                                             int32_t max_len, void *out, int32_t *status_word,
                                             void *stream) {
    using namespace zipvl;
    const char *who = "zipvl_decode_noalloc";
    if (!d) return fail(ZIPVL_ERR_INVALID_ARG, "%s: desc is NULL", who);
    if (d->batch < 1 || d->batch > 65535 || d->n_q_heads < 1 || d->n_kv_heads < 1 ||
        d->n_q_heads % d->n_kv_heads)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: batch %d heads %d / %d", who, d->batch,
                    d->n_q_heads, d->n_kv_heads);
    if ((d->dtype != ZIPVL_BF16 && d->dtype != ZIPVL_F32 && d->dtype != ZIPVL_F16) ||
        (d->head_dim != 64 && d->head_dim != 96 && d->head_dim != 128) ||
        (d->n_q_heads / d->n_kv_heads > 8 && !decode_tc_supported(*d)))
        return fail(ZIPVL_ERR_UNSUPPORTED, "%s: dtype %d head_dim %d group %d", who, d->dtype,
                    d->head_dim, d->n_q_heads / d->n_kv_heads);
    if (!q || !k_cache || !v_cache || !cache_off || !capacity || !seq_lens || !out)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: NULL pointer", who);
    if ((k_new == NULL) != (v_new == NULL))
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: k_new and v_new must both be given or both NULL", who);
    if (max_len < 1) return fail(ZIPVL_ERR_INVALID_ARG, "%s: max_len = %d", who, max_len);
    if (!(d->softmax_scale >= 0.f) || isinf(d->softmax_scale))
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: softmax_scale", who);
    if (((uintptr_t)q | (uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)out) & 15u)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: tensors must be 16-byte aligned", who);
    const size_t need = decode_ws_bytes(d->batch, d->n_q_heads, d->head_dim, max_len, d->n_kv_heads, d->dtype);
    if (need > kNoAllocScratchBytes)
        return fail(ZIPVL_ERR_WORKSPACE,
                    "%s: batch %d x %d heads x max_len %d needs %zu bytes of scratch, the built-in "
                    "scratch holds %zu; use zipvl_decode with a workspace instead",
                    who, d->batch, d->n_q_heads, max_len, need, (size_t)kNoAllocScratchBytes);
    void *scratch = nullptr;
    const zipvl_status s = noalloc_scratch(&scratch);
    if (s != ZIPVL_OK) return s;
    const float scale = d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / sqrtf((float)d->head_dim);
    return launch_decode(*d, scale * kLog2e, q, k_new, v_new, k_cache, v_cache, cache_off, capacity,
                         seq_lens, max_len, out, scratch, status_word, (cudaStream_t)stream);
}


// ---- decode over a paged cache -------------------------------------------------
extern "C" zipvl_status zipvl_decode_paged(const zipvl_decode_desc *d, const void *q,
                                           const void *k_new, const void *v_new, void *k_pages,
                                           void *v_pages, const int32_t *block_table,
                                           int32_t table_stride, int32_t page_rows, int32_t n_pages,
                                           const int32_t *capacity, int32_t *seq_lens,
                                           int32_t max_len, void *out, void *ws, size_t ws_bytes,
                                           int32_t *status_word, void *stream) {
    using namespace zipvl;
    const char *who = "zipvl_decode_paged";
    if (!d) return fail(ZIPVL_ERR_INVALID_ARG, "%s: desc is NULL", who);
    if (d->batch < 1 || d->batch > 65535 || d->n_q_heads < 1 || d->n_kv_heads < 1 ||
        d->n_q_heads % d->n_kv_heads)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: batch %d heads %d / %d", who, d->batch,
                    d->n_q_heads, d->n_kv_heads);
    if ((d->dtype != ZIPVL_BF16 && d->dtype != ZIPVL_F32 && d->dtype != ZIPVL_F16) ||
        (d->head_dim != 64 && d->head_dim != 96 && d->head_dim != 128) ||
        (d->n_q_heads / d->n_kv_heads > 8 && !decode_tc_supported(*d)))
        return fail(ZIPVL_ERR_UNSUPPORTED, "%s: dtype %d head_dim %d group %d", who, d->dtype,
                    d->head_dim, d->n_q_heads / d->n_kv_heads);
    if (!q || !k_pages || !v_pages || !block_table || !capacity || !seq_lens || !out || !ws)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: NULL pointer", who);
    if ((k_new == NULL) != (v_new == NULL))
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: k_new and v_new must both be given or both NULL", who);
    if (max_len < 1) return fail(ZIPVL_ERR_INVALID_ARG, "%s: max_len = %d", who, max_len);
    int shift = 0;
    while ((1 << shift) < page_rows) ++shift;
    if (page_rows < 16 || page_rows > 1024 || (1 << shift) != page_rows)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: page_rows = %d (a power of two from 16 to 1024)", who, page_rows);
    if (n_pages < 1 || table_stride < (max_len + page_rows - 1) / page_rows)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: n_pages = %d, table_stride = %d for max_len %d", who,
                    n_pages, table_stride, max_len);
    if (!(d->softmax_scale >= 0.f) || isinf(d->softmax_scale))
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: softmax_scale", who);
    if (((uintptr_t)q | (uintptr_t)k_pages | (uintptr_t)v_pages | (uintptr_t)out | (uintptr_t)ws) & 15u)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: tensors must be 16-byte aligned", who);
    const size_t need = (decode_ws_bytes(d->batch, d->n_q_heads, d->head_dim, max_len, d->n_kv_heads, d->dtype) + 255) & ~(size_t)255;
    if (ws_bytes < need) return fail(ZIPVL_ERR_WORKSPACE, "%s: workspace %zu < %zu", who, ws_bytes, need);
    const float scale = d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / sqrtf((float)d->head_dim);
    return dispatch_decode(*d, scale * kLog2e, q, k_new, v_new, k_pages, v_pages, nullptr,
                           PageArgs{block_table, table_stride, shift, n_pages}, capacity, seq_lens,
                           max_len, out, ws, status_word, (cudaStream_t)stream);
}
