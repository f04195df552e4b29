// Probe scoring on CUDA cores: exact fp32 FMA path (fp32 tensors) and the
// general-shape path for bf16 / fp16.  Supplementary Eq. A with the causal mask of
// Eq. 2, column sums of Eq. 6, normalisation of Eq. 8.
//
// A column sum of a row-softmax needs every row's final max and denominator,
// so the contraction runs twice and the attention matrix never leaves the SM:
//   pass 1  one thread per probe row, keys streamed through shared memory:
//           per (head, key chunk, probe) running max m and sum l (base 2);
//   pass 2  one thread per key, probe rows streamed through shared memory:
//           column sum of exp2(s - m_r) / l_r over the probes that see the key;
//   pass 3  sum over heads in fixed order, nnz by binary search, normalise.
// Nothing uses float atomics, so results repeat bit for bit.
#include "common.cuh"

namespace zipvl {
namespace {

constexpr int kChunk = 256;   // keys per pass-1 block
constexpr int kKeyTile = 32;  // keys staged in shared memory at a time
constexpr int kProbeTile = 32;
constexpr int kThreads = 128;

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
score_stats_kernel(LayerArgs a, const T *__restrict__ q, const T *__restrict__ k,
                   const int32_t *__restrict__ probe_pos, int P, int n_chunks,
                   float2 *__restrict__ stats, int32_t *status_word) {
    __shared__ __align__(16) float Ks[kKeyTile][D];
    const int chunk = blockIdx.x, h = blockIdx.y, g = h / a.G;
    const int r = blockIdx.z * kThreads + threadIdx.x;
    const int j0 = chunk * kChunk, j1 = min(a.L, j0 + kChunk);

    int c = -1;
    if (r < P) {
        c = probe_pos[r];
        if (c < 0 || c >= a.L) {
            if (chunk == 0 && h == 0) report(status_word, ZIPVL_DEV_BAD_INDEX);
            c = -1;
        }
    }
    float qr[D];
    if (c >= 0) {
        const T *qp = q + (long long)c * a.q_stride + (long long)h * D;
#pragma unroll
        for (int t = 0; t < D; t += 8) {
            float x[8];
            load8(qp + t, x);
#pragma unroll
            for (int u = 0; u < 8; ++u) qr[t + u] = x[u] * a.scale_log2;
        }
    } else {
#pragma unroll
        for (int t = 0; t < D; ++t) qr[t] = 0.f;
    }

    float m = -INFINITY, l = 0.f;
    for (int jt = j0; jt < j1; jt += kKeyTile) {
        __syncthreads();
        // stage keys jt .. jt+31 of kv head g as floats
        for (int e = threadIdx.x; e < kKeyTile * (D / 8); e += kThreads) {
            const int row = e / (D / 8), col = (e % (D / 8)) * 8;
            float x[8];
            if (jt + row < j1) {
                load8(k + (long long)(jt + row) * a.kv_stride + (long long)g * D + col, x);
            } else {
#pragma unroll
                for (int u = 0; u < 8; ++u) x[u] = 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) Ks[row][col + u] = x[u];
        }
        __syncthreads();
        const int jend = min(min(j1, jt + kKeyTile), c + 1);  // causal: keys <= c
        for (int j = jt; j < jend; ++j) {
            const float4 *kr = reinterpret_cast<const float4 *>(Ks[j - jt]);
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
            for (int t = 0; t < D / 4; ++t) {
                const float4 kv = kr[t];
                s0 = fmaf(qr[4 * t], kv.x, s0);
                s1 = fmaf(qr[4 * t + 1], kv.y, s1);
                s2 = fmaf(qr[4 * t + 2], kv.z, s2);
                s3 = fmaf(qr[4 * t + 3], kv.w, s3);
            }
            const float s = (s0 + s1) + (s2 + s3);
            if (s > m) {
                l *= fast_exp2(m - s);
                m = s;
            }
            l += fast_exp2(s - m);
        }
    }
    if (r < P) stats[((long long)h * n_chunks + chunk) * P + r] = make_float2(m, l);
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
score_colsum_kernel(LayerArgs a, const T *__restrict__ q, const T *__restrict__ k,
                    const int32_t *__restrict__ probe_pos, int P, int n_chunks,
                    const float2 *__restrict__ stats, float *__restrict__ partial) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *Qs = reinterpret_cast<float *>(smem_raw);      // [kProbeTile][D]
    float *Ms = Qs + kProbeTile * D;                       // [P] merged row max
    float *Il = Ms + P;                                    // [P] 1 / merged row sum
    int *Pos = reinterpret_cast<int *>(Il + P);            // [P]

    const int h = blockIdx.y, g = h / a.G;
    const int jb = blockIdx.x * kThreads, j = jb + threadIdx.x;

    // merge the per-chunk row statistics of this head
    for (int r = threadIdx.x; r < P; r += kThreads) {
        int c = probe_pos[r];
        if (c < 0 || c >= a.L) c = -1;
        Pos[r] = c;
        float M = -INFINITY;
        for (int ch = 0; ch < n_chunks; ++ch)
            M = fmaxf(M, stats[((long long)h * n_chunks + ch) * P + r].x);
        float Lsum = 0.f;
        for (int ch = 0; ch < n_chunks; ++ch) {
            const float2 s = stats[((long long)h * n_chunks + ch) * P + r];
            if (s.y > 0.f) Lsum += s.y * fast_exp2(s.x - M);
        }
        Ms[r] = M;
        Il[r] = Lsum > 0.f ? 1.f / Lsum : 0.f;
    }

    float kr[D];
    if (j < a.L) {
        const T *kp = k + (long long)j * a.kv_stride + (long long)g * D;
#pragma unroll
        for (int t = 0; t < D; t += 8) {
            float x[8];
            load8(kp + t, x);
#pragma unroll
            for (int u = 0; u < 8; ++u) kr[t + u] = x[u] * a.scale_log2;
        }
    } else {
#pragma unroll
        for (int t = 0; t < D; ++t) kr[t] = 0.f;
    }
    __syncthreads();

    float colsum = 0.f;
    for (int rt = 0; rt < P; rt += kProbeTile) {
        const int rend = min(P, rt + kProbeTile);
        // if every probe of the tile sits before this block's first key, no key
        // of the block is visible to the tile (uniform over the block)
        int tile_max = -1;
        for (int r = rt; r < rend; ++r) tile_max = max(tile_max, Pos[r]);
        if (tile_max < jb) continue;
        __syncthreads();
        for (int e = threadIdx.x; e < kProbeTile * (D / 8); e += kThreads) {
            const int row = e / (D / 8), col = (e % (D / 8)) * 8;
            float x[8];
            const int c = (rt + row < P) ? Pos[rt + row] : -1;
            if (c >= 0) {
                load8(q + (long long)c * a.q_stride + (long long)h * D + col, x);
            } else {
#pragma unroll
                for (int u = 0; u < 8; ++u) x[u] = 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) Qs[row * D + col + u] = x[u];
        }
        __syncthreads();
        for (int r = rt; r < rend; ++r) {
            if (Pos[r] < j) continue;       // causal mask (also skips invalid probes)
            const float4 *qv = reinterpret_cast<const float4 *>(Qs + (r - rt) * D);
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
            for (int t = 0; t < D / 4; ++t) {
                const float4 x = qv[t];
                s0 = fmaf(kr[4 * t], x.x, s0);
                s1 = fmaf(kr[4 * t + 1], x.y, s1);
                s2 = fmaf(kr[4 * t + 2], x.z, s2);
                s3 = fmaf(kr[4 * t + 3], x.w, s3);
            }
            const float s = (s0 + s1) + (s2 + s3);
            colsum += fast_exp2(s - Ms[r]) * Il[r];
        }
    }
    if (j < a.L) partial[(long long)h * a.L + j] = colsum;
}

// first r with probe_pos[r] >= x (probe_pos ascending)
__device__ __forceinline__ int lower_bound(const int32_t *p, int n, int x) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (p[mid] < x) lo = mid + 1; else hi = mid;
    }
    return lo;
}

__global__ void score_finalize_kernel(int L, int Hq, int P, const float *__restrict__ partial,
                                      const int32_t *__restrict__ probe_pos,
                                      float *__restrict__ acc, float *__restrict__ norm) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= L) return;
    float s = 0.f;
    for (int h = 0; h < Hq; ++h) s += partial[(long long)h * L + j];
    // structural nnz: probes at positions j .. L-1
    const int nnz = lower_bound(probe_pos, P, L) - lower_bound(probe_pos, P, j);
    acc[j] = s;
    norm[j] = nnz > 0 ? s / ((float)Hq * (float)nnz) : 0.f;
}

}  // namespace

__global__ void sum_to_double_kernel(int L, const float *__restrict__ x, double *__restrict__ out) {
    __shared__ double sh[1024];
    double s = 0.0;
    for (int j = threadIdx.x; j < L; j += blockDim.x) s += (double)x[j];
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int w = blockDim.x / 2; w > 0; w >>= 1) {
        if ((int)threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = sh[0];
}

size_t score_simt_ws_bytes(int L, int Hq, int P) {
    const size_t n_chunks = (L + kChunk - 1) / kChunk;
    size_t stats = (size_t)Hq * n_chunks * P * sizeof(float2);
    stats = (stats + 255) & ~(size_t)255;
    return stats + (size_t)Hq * L * sizeof(float);
}

template <typename T, int D>
static zipvl_status run(const LayerArgs &a, const void *q, const void *k,
                        const int32_t *probe_pos, int P, float *acc, float *norm, double *total,
                        void *ws, int32_t *status_word, cudaStream_t st) {
    const int n_chunks = (a.L + kChunk - 1) / kChunk;
    size_t stats_bytes = (size_t)a.Hq * n_chunks * P * sizeof(float2);
    stats_bytes = (stats_bytes + 255) & ~(size_t)255;
    float2 *stats = reinterpret_cast<float2 *>(ws);
    float *partial = reinterpret_cast<float *>(reinterpret_cast<char *>(ws) + stats_bytes);

    dim3 g1(n_chunks, a.Hq, (P + kThreads - 1) / kThreads);
    score_stats_kernel<T, D><<<g1, kThreads, 0, st>>>(a, (const T *)q, (const T *)k, probe_pos, P,
                                                     n_chunks, stats, status_word);
    const size_t smem = (size_t)kProbeTile * D * sizeof(float) + (size_t)P * 12;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(score_colsum_kernel<T, D>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "score: smem opt-in: %s", cudaGetErrorString(e));
    }
    dim3 g2((a.L + kThreads - 1) / kThreads, a.Hq);
    score_colsum_kernel<T, D><<<g2, kThreads, smem, st>>>(a, (const T *)q, (const T *)k, probe_pos,
                                                         P, n_chunks, stats, partial);
    score_finalize_kernel<<<(a.L + 255) / 256, 256, 0, st>>>(a.L, a.Hq, P, partial, probe_pos, acc,
                                                            norm);
    if (total) sum_to_double_kernel<<<1, 1024, 0, st>>>(a.L, acc, total);
    count_launches(total ? 4 : 3);
    return check_launch("zipvl_score");
}

zipvl_status launch_score_simt(const LayerArgs &a, int dtype, const void *q, const void *k,
                               const int32_t *probe_pos, int P, float *acc, float *norm,
                               double *total, void *ws, int32_t *status_word, cudaStream_t st) {
    if (P > 8192) return fail(ZIPVL_ERR_UNSUPPORTED, "score: n_probe %d > 8192", P);
    if (dtype == ZIPVL_F32) {
        if (a.D == 64) return run<float, 64>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
        if (a.D == 96) return run<float, 96>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
        if (a.D == 128) return run<float, 128>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
    } else if (dtype == ZIPVL_F16) {
        if (a.D == 64) return run<__half, 64>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
        if (a.D == 96) return run<__half, 96>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
        if (a.D == 128) return run<__half, 128>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
    } else {
        if (a.D == 64) return run<__nv_bfloat16, 64>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
        if (a.D == 96) return run<__nv_bfloat16, 96>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
        if (a.D == 128) return run<__nv_bfloat16, 128>(a, q, k, probe_pos, P, acc, norm, total, ws, status_word, st);
    }
    return fail(ZIPVL_ERR_UNSUPPORTED, "score: head_dim %d", a.D);
}

}  // namespace zipvl
