// Sparse causal prefill attention on CUDA cores (Algorithm 1, attention over
// Q[T], K[T], V[T]; Eq. 2 on the gathered tokens): the exact-fp32 path for
// fp32 tensors and the general-shape path for bf16 / fp16.  The tensor-core kernel in
// prefill_tc.cu takes over for the 16-bit shapes it supports.
//
// One CTA = 64 gathered query rows of one head, 8 warps x 8 rows.  Keys and
// values of the kept tokens are gathered by index, 32 at a time, into shared
// memory as floats; lane j of a warp scores key j for the warp's rows, the
// online softmax (base 2) runs across the lanes, and each lane owns d/32
// output channels.  PADDED output: the CTA that owns row i also zero-fills the
// rows of the dropped tokens between T[i-1] and T[i] (and after the last kept
// token), so padding costs no extra launch.
#include "common.cuh"

namespace zipvl {
namespace {

constexpr int kBM = 64, kBN = 32, kPfThreads = 256, kRows = 8;

template <typename T, int D>
__global__ void __launch_bounds__(kPfThreads)
prefill_simt_kernel(LayerArgs a, const T *__restrict__ q, const T *__restrict__ k,
                    const T *__restrict__ v, const int32_t *__restrict__ idx,
                    const int32_t *__restrict__ k_dev, int k_max, T *__restrict__ out,
                    int out_mode, int32_t *status_word) {
    constexpr int KP = D + 4;   // padded key row: conflict-free float4 reads by 8 lanes
    constexpr int CPL = D / 32; // output channels per lane
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *Qs = reinterpret_cast<float *>(smem_raw);  // [kBM][D], pre-scaled
    float *Ks = Qs + kBM * D;                          // [kBN][KP]
    float *Vs = Ks + kBN * KP;                         // [kBN][D]

    int n = *k_dev;
    if (n > k_max || n < 0) {
        if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0)
            report(status_word, ZIPVL_DEV_CAPACITY);
        n = n < 0 ? 0 : k_max;
    }
    const int h = blockIdx.y, g = h / a.G;
    const int i0 = blockIdx.x * kBM;
    if (n == 0 && blockIdx.x == 0 && out_mode == ZIPVL_OUT_PADDED) {
        // nothing kept: every row is a dropped token's row
        for (long long e = threadIdx.x; e < (long long)a.L * D; e += kPfThreads)
            store_elem(out + ((e / D) * a.Hq + h) * D + (e % D), 0.f);
    }
    if (i0 >= n) return;
    const int i1 = min(n, i0 + kBM);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // stage the query rows (scaled by softmax_scale * log2 e)
    for (int e = threadIdx.x; e < kBM * (D / 8); e += kPfThreads) {
        const int row = e / (D / 8), col = (e % (D / 8)) * 8;
        float x[8];
        int t = (i0 + row < i1) ? idx[i0 + row] : -1;
        if (i0 + row < i1 && (t < 0 || t >= a.L)) { report(status_word, ZIPVL_DEV_BAD_INDEX); t = -1; }
        if (t >= 0) {
            load8(q + (long long)t * a.q_stride + (long long)h * D + col, x);
        } else {
#pragma unroll
            for (int u = 0; u < 8; ++u) x[u] = 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) Qs[row * D + col + u] = x[u] * a.scale_log2;
    }

    float m[kRows], l[kRows], o[kRows][CPL];
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        m[r] = -INFINITY;
        l[r] = 0.f;
#pragma unroll
        for (int c = 0; c < CPL; ++c) o[r][c] = 0.f;
    }

    const int row_base = i0 + warp * kRows;  // first gathered row of this warp
    for (int jt = 0; jt < i1; jt += kBN) {
        __syncthreads();
        for (int e = threadIdx.x; e < kBN * (D / 8); e += kPfThreads) {
            const int row = e / (D / 8), col = (e % (D / 8)) * 8;
            float x[8], y[8];
            int t = (jt + row < i1) ? idx[jt + row] : -1;
            if (t < 0 || t >= a.L) t = -1;
            if (t >= 0) {
                const long long off = (long long)t * a.kv_stride + (long long)g * D + col;
                load8(k + off, x);
                load8(v + off, y);
            } else {
#pragma unroll
                for (int u = 0; u < 8; ++u) { x[u] = 0.f; y[u] = 0.f; }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) { Ks[row * KP + col + u] = x[u]; Vs[row * D + col + u] = y[u]; }
        }
        __syncthreads();
        if (jt > row_base + kRows - 1) continue;  // whole tile is above this warp's diagonal

        // scores of key (jt + lane) for the warp's 8 rows
        float s[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) s[r] = 0.f;
        const float4 *kr = reinterpret_cast<const float4 *>(Ks + lane * KP);
#pragma unroll 4
        for (int t = 0; t < D / 4; ++t) {
            const float4 kv = kr[t];
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                const float4 qv = *reinterpret_cast<const float4 *>(Qs + (warp * kRows + r) * D + 4 * t);
                s[r] = fmaf(qv.x, kv.x, s[r]);
                s[r] = fmaf(qv.y, kv.y, s[r]);
                s[r] = fmaf(qv.z, kv.z, s[r]);
                s[r] = fmaf(qv.w, kv.w, s[r]);
            }
        }
        const int j = jt + lane;
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const int i = row_base + r;
            const bool vis = (j <= i) && (i < i1);  // causal inside T; j <= i < n
            float sv = vis ? s[r] : -INFINITY;
            float mx = sv;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            const float mn = fmaxf(m[r], mx);
            float p = 0.f, sc = 1.f;
            if (mn != -INFINITY) {
                sc = fast_exp2(m[r] - mn);
                p = fast_exp2(sv - mn);
            }
            float ps = p;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
            m[r] = mn;
            l[r] = l[r] * sc + ps;
#pragma unroll
            for (int c = 0; c < CPL; ++c) o[r][c] *= sc;
            s[r] = p;
        }
        // o[r][c] += sum_j p[r][j] * V[j][lane + 32 c]
        for (int jj = 0; jj < kBN; ++jj) {
            float vv[CPL];
#pragma unroll
            for (int c = 0; c < CPL; ++c) vv[c] = Vs[jj * D + lane + 32 * c];
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                const float p = __shfl_sync(0xffffffffu, s[r], jj);
#pragma unroll
                for (int c = 0; c < CPL; ++c) o[r][c] = fmaf(p, vv[c], o[r][c]);
            }
        }
    }

    // write the rows; PADDED also zero-fills the dropped tokens owned by each row
#pragma unroll
    for (int r = 0; r < kRows; ++r) {
        const int i = row_base + r;
        if (i >= i1) continue;
        const int t = idx[i];
        if (t < 0 || t >= a.L) continue;
        const float inv = l[r] > 0.f ? 1.f / l[r] : 0.f;
        const long long orow = (out_mode == ZIPVL_OUT_PADDED) ? t : i;
        T *dst = out + (orow * a.Hq + h) * D;
#pragma unroll
        for (int c = 0; c < CPL; ++c) store_elem(dst + lane + 32 * c, o[r][c] * inv);
        if (out_mode == ZIPVL_OUT_PADDED) {
            // the gap in front of this token; a previous entry that is out of range or not
            // below this one (the list must ascend) is read as "no gap"
            int lo = 0;
            if (i > 0) {
                const int tp = idx[i - 1];
                lo = (tp >= 0 && tp < t) ? tp + 1 : t;
            }
            for (int z = lo; z < t; ++z) {
                T *zr = out + ((long long)z * a.Hq + h) * D;
#pragma unroll
                for (int c = 0; c < CPL; ++c) store_elem(zr + lane + 32 * c, 0.f);
            }
            if (i == n - 1) {
                for (int z = t + 1; z < a.L; ++z) {
                    T *zr = out + ((long long)z * a.Hq + h) * D;
#pragma unroll
                    for (int c = 0; c < CPL; ++c) store_elem(zr + lane + 32 * c, 0.f);
                }
            }
        }
    }
}

template <typename T, int D>
zipvl_status run(const LayerArgs &a, const void *q, const void *k, const void *v,
                 const int32_t *idx, const int32_t *k_dev, int k_max, void *out, int out_mode,
                 int32_t *status_word, cudaStream_t st) {
    const size_t smem = (size_t)(kBM * D + kBN * (D + 4) + kBN * D) * sizeof(float) + kBN * sizeof(int);
    cudaError_t e = cudaFuncSetAttribute(prefill_simt_kernel<T, D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "sparse_prefill: smem opt-in: %s", cudaGetErrorString(e));
    dim3 grid((k_max + kBM - 1) / kBM, a.Hq);
    prefill_simt_kernel<T, D><<<grid, kPfThreads, smem, st>>>(
        a, (const T *)q, (const T *)k, (const T *)v, idx, k_dev, k_max, (T *)out, out_mode,
        status_word);
    count_launches(1);
    return check_launch("zipvl_sparse_prefill");
}

}  // namespace

zipvl_status launch_prefill_simt(const LayerArgs &a, int dtype, const void *q, const void *k,
                                 const void *v, const int32_t *idx, const int32_t *k_dev,
                                 int k_max, void *out, int out_mode, int32_t *status_word,
                                 cudaStream_t st) {
    if (dtype == ZIPVL_F32) {
        if (a.D == 64) return run<float, 64>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
        if (a.D == 96) return run<float, 96>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
        if (a.D == 128) return run<float, 128>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
    } else if (dtype == ZIPVL_F16) {
        if (a.D == 64) return run<__half, 64>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
        if (a.D == 96) return run<__half, 96>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
        if (a.D == 128) return run<__half, 128>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
    } else {
        if (a.D == 64) return run<__nv_bfloat16, 64>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
        if (a.D == 96) return run<__nv_bfloat16, 96>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
        if (a.D == 128) return run<__nv_bfloat16, 128>(a, q, k, v, idx, k_dev, k_max, out, out_mode, status_word, st);
    }
    return fail(ZIPVL_ERR_UNSUPPORTED, "sparse_prefill: head_dim %d", a.D);
}

}  // namespace zipvl
