// Mixed-precision KV cache (Sec. 4.3, Table 3: the tokens of T at 4 bits, the others at 2)
// and the decode step over it (Algorithm 2, Eq. 4-5, with the rows dequantised on the fly).
//
// The paper takes the quantiser from the work it cites and fixes only the bit allocation.
// The reading built here: no token is evicted; keys and values are quantised per (token,
// KV head) over the head_dim channels with an asymmetric uniform quantiser,
//     scale = (max - min) / (2^b - 1),  code = clip(rint((x - min) * (1 / scale)), 0, 2^b - 1),
// scale and min rounded to the storage type and kept beside the codes; every step that
// decides a code is a single correctly rounded fp32 operation, so the codes are the same
// bits as the CPU checker's.  Softmax attention does not depend on the order of the cached
// rows, so the cache is two blocks: "hi" (the tokens of T, in T's order; decoded tokens are
// appended here) and "lo" (the others, ascending).  Codes are packed little-end first
// (channel c in byte c*b/8 at bit (c*b)%8); a row of a block is Hkv * d*b/8 bytes; the
// parameters of a block are [rows, Hkv, 4] storage-type values (k scale, k min, v scale, v min).
#include <math.h>

#include "common.cuh"

namespace zipvl {
namespace {

constexpr int kQuantThreads = 256;
constexpr int kQuantIters = 8;      // (token, head) pairs per lane group and CTA

template <bool kHalf>
__device__ __forceinline__ float storage_round(float x, unsigned short *bits) {
    if (kHalf) {
        const __half h = __float2half_rn(x);
        *bits = __half_as_ushort(h);
        return __half2float(h);
    }
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    *bits = __bfloat16_as_ushort(h);
    return __bfloat162float(h);
}
template <bool kHalf>
__device__ __forceinline__ float storage_to_float(unsigned short bits) {
    return kHalf ? __half2float(__ushort_as_half(bits)) : __bfloat162float(__ushort_as_bfloat16(bits));
}
template <bool kHalf>
__device__ __forceinline__ void unpack8s(const uint4 r, float (&x)[8]) {
    if (kHalf) unpack8h(r, x);
    else unpack8(r, x);
}

// One (row, head) group of kLanes adjacent lanes, eight channels per lane: the quantiser's
// parameters (rounded to the storage type) and this lane's eight codes packed at `bits` each.
template <bool kHalf, int kLanes>
__device__ __forceinline__ uint32_t quantise8(const float (&x)[8], int bits, unsigned short *scale_bits,
                                              unsigned short *zero_bits) {
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int e = 1; e < 8; ++e) { mn = fminf(mn, x[e]); mx = fmaxf(mx, x[e]); }
#pragma unroll
    for (int o = kLanes / 2; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    const float levels = (float)((1 << bits) - 1);
    const float scale = storage_round<kHalf>(__fdiv_rn(__fsub_rn(mx, mn), levels), scale_bits);
    const float zero = storage_round<kHalf>(mn, zero_bits);
    uint32_t packed = 0;
    if (scale > 0.f) {
        const float inv = __frcp_rn(scale);             // one correctly rounded reciprocal per row
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float c = fminf(fmaxf(rintf(__fmul_rn(__fsub_rn(x[e], zero), inv)), 0.f), levels);
            packed |= (uint32_t)c << (bits * e);
        }
    }
    return packed;
}

// Writes one lane's eight codes (32 bits at 4 bits each, 16 at 2) and, from the group's first
// lane, the four parameters of the (row, head).
__device__ __forceinline__ void store_codes(unsigned char *row_base, int lane_in_group, int bits, uint32_t packed) {
    if (bits == 4) reinterpret_cast<uint32_t *>(row_base)[lane_in_group] = packed;
    else reinterpret_cast<unsigned short *>(row_base)[lane_in_group] = (unsigned short)packed;
}

struct QuantBlocks {
    unsigned char *k_hi, *v_hi, *k_lo, *v_lo;
    unsigned short *p_hi, *p_lo;      // [rows, Hkv, 4] storage-type bits
    int cap_hi, cap_lo;
};

// The blocks of request b: the call's own (one request) or entry b of the caller's device table.
// A table entry cannot be checked on the host: one with a NULL or misaligned block or a capacity
// below 1 is reported and its request skipped (no append, an output of zeros).
__device__ __forceinline__ bool request_blocks(const zipvl_quant_cache *caches, int b, QuantBlocks &qb,
                                               int32_t *&lens) {
    if (caches == nullptr) return true;
    const zipvl_quant_cache c = caches[b];
    qb = QuantBlocks{(unsigned char *)c.k_hi, (unsigned char *)c.v_hi, (unsigned char *)c.k_lo, (unsigned char *)c.v_lo,
                     (unsigned short *)c.params_hi, (unsigned short *)c.params_lo, c.cap_hi, c.cap_lo};
    lens = c.lens;
    const unsigned long long all = (unsigned long long)c.k_hi | (unsigned long long)c.v_hi | (unsigned long long)c.k_lo |
                                   (unsigned long long)c.v_lo | (unsigned long long)c.params_hi |
                                   (unsigned long long)c.params_lo;
    return c.k_hi && c.v_hi && c.k_lo && c.v_lo && c.params_hi && c.params_lo && c.lens && !(all & 15ull) &&
           !((unsigned long long)c.lens & 3ull) && c.cap_hi >= 1 && c.cap_lo >= 1;
}

template <bool kHalf, int D>
__global__ void __launch_bounds__(kQuantThreads)
quantize_kv_kernel(LayerArgs a, const unsigned short *__restrict__ k, const unsigned short *__restrict__ v,
                   const int32_t *__restrict__ idx, const int32_t *__restrict__ k_dev, int k_max,
                   QuantBlocks qb, int32_t *__restrict__ lens_out, int32_t *status_word) {
    constexpr int kLanes = D / 8;                 // lanes per (token, head)
    constexpr int kGroups = 32 / kLanes;          // groups per warp
    grid_launch_dependents();
    grid_dependency_wait(k, v, idx, k_dev);       // T and k are the selection's output
    int n = *k_dev;
    if (n > k_max || n < 0) {
        if (blockIdx.x == 0 && threadIdx.x == 0) report(status_word, ZIPVL_DEV_CAPACITY);
        n = n < 0 ? 0 : k_max;
    }
    if (n > qb.cap_hi || a.L - n > qb.cap_lo) {
        if (blockIdx.x == 0 && threadIdx.x == 0) report(status_word, ZIPVL_DEV_CAPACITY);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        lens_out[0] = min(n, qb.cap_hi);
        lens_out[1] = min(a.L - n, qb.cap_lo);
    }
    // A CTA takes kPairsPerCta consecutive (token, head) pairs, i.e. a short run of tokens.
    // Where each of those tokens goes -- row i of the 4-bit block if it is T's i-th entry, else
    // row (t - #entries of T below t) of the 2-bit block -- is looked up once per token (a
    // binary search in the ascending list) by the first threads and shared.
    constexpr int kPairsPerIter = (kQuantThreads / 32) * kGroups;
    constexpr int kPairsPerCta = kPairsPerIter * kQuantIters;
    __shared__ int s_row[kPairsPerCta + 2];            // >= 0: hi row; < 0: -(lo row) - 1
    const int lane = threadIdx.x & 31, lg = lane % kLanes;
    const long long n_pairs = (long long)a.L * a.Hkv;
    const long long p0 = (long long)blockIdx.x * kPairsPerCta;
    const int t_first = (int)(p0 / a.Hkv);
    const int t_last = (int)(min(p0 + kPairsPerCta, n_pairs) - 1) / a.Hkv;
    for (int t = t_first + (int)threadIdx.x; t <= t_last; t += kQuantThreads) {
        int lo = 0, hi = n;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (idx[mid] < t) lo = mid + 1; else hi = mid;
        }
        s_row[t - t_first] = (lo < n && idx[lo] == t) ? lo : -(t - lo) - 1;
    }
    __syncthreads();
#pragma unroll 2
    for (int it = 0; it < kQuantIters; ++it) {
        const long long p = p0 + (long long)it * kPairsPerIter + (threadIdx.x >> 5) * kGroups + lane / kLanes;
        const bool live = p < n_pairs;
        const int t = live ? (int)(p / a.Hkv) : t_first, g = live ? (int)(p % a.Hkv) : 0;
        const int where = s_row[t - t_first];
        const bool in_T = where >= 0;
        const int bits = in_T ? 4 : 2;
        const int row = in_T ? where : -where - 1;         // its row in the "hi" / "lo" block
        const bool fits = live && row < (in_T ? qb.cap_hi : qb.cap_lo);
        float xk[8], xv[8];
        if (live) {
            const long long off = (long long)t * a.kv_stride + (long long)g * D + lg * 8;
            unpack8s<kHalf>(*reinterpret_cast<const uint4 *>(k + off), xk);
            unpack8s<kHalf>(*reinterpret_cast<const uint4 *>(v + off), xv);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) { xk[e] = 0.f; xv[e] = 0.f; }
        }
        unsigned short ks, kz, vs, vz;
        const uint32_t ck = quantise8<kHalf, kLanes>(xk, bits, &ks, &kz);
        const uint32_t cv = quantise8<kHalf, kLanes>(xv, bits, &vs, &vz);
        if (fits) {
            const long long rh = (long long)row * a.Hkv + g;
            const int row_bytes = D * bits / 8;
            store_codes((in_T ? qb.k_hi : qb.k_lo) + rh * row_bytes, lg, bits, ck);
            store_codes((in_T ? qb.v_hi : qb.v_lo) + rh * row_bytes, lg, bits, cv);
            if (lg == 0) {
                unsigned short *pp = (in_T ? qb.p_hi : qb.p_lo) + rh * 4;
                *reinterpret_cast<uint2 *>(pp) = make_uint2((uint32_t)ks | ((uint32_t)kz << 16),
                                                            (uint32_t)vs | ((uint32_t)vz << 16));
            }
        }
    }
}

// Eq. 4 on the quantised cache: the new token's key and value, quantised at 4 bits, become
// row lens[0] of the "hi" block; lens[0] += 1.  One CTA per request, one lane group per KV head.
template <bool kHalf, int D>
__global__ void __launch_bounds__(1024)
quant_append_kernel(int Hkv, const unsigned short *__restrict__ k_new, const unsigned short *__restrict__ v_new,
                    QuantBlocks qb, int32_t *lens, const zipvl_quant_cache *__restrict__ caches,
                    int32_t *status_word) {
    constexpr int kLanes = D / 8;
    grid_launch_dependents();
    grid_dependency_wait(k_new, v_new, lens, caches);
    const int b = blockIdx.x;
    if (!request_blocks(caches, b, qb, lens)) {
        if (threadIdx.x == 0) report(status_word, ZIPVL_DEV_BAD_INDEX);
        return;
    }
    k_new += (long long)b * Hkv * D;
    v_new += (long long)b * Hkv * D;
    const int n_hi = lens[0];
    const bool room = n_hi >= 0 && n_hi < qb.cap_hi;
    const int grp = threadIdx.x / kLanes, lg = threadIdx.x % kLanes;
    const bool live = grp < Hkv;
    float xk[8], xv[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { xk[e] = 0.f; xv[e] = 0.f; }
    if (live) {
        unpack8s<kHalf>(*reinterpret_cast<const uint4 *>(k_new + (long long)grp * D + lg * 8), xk);
        unpack8s<kHalf>(*reinterpret_cast<const uint4 *>(v_new + (long long)grp * D + lg * 8), xv);
    }
    unsigned short ks, kz, vs, vz;
    const uint32_t ck = quantise8<kHalf, kLanes>(xk, 4, &ks, &kz);
    const uint32_t cv = quantise8<kHalf, kLanes>(xv, 4, &vs, &vz);
    if (live && room) {
        const long long rh = (long long)n_hi * Hkv + grp;
        store_codes(qb.k_hi + rh * (D / 2), lg, 4, ck);
        store_codes(qb.v_hi + rh * (D / 2), lg, 4, cv);
        if (lg == 0)
            *reinterpret_cast<uint2 *>(qb.p_hi + rh * 4) =
                make_uint2((uint32_t)ks | ((uint32_t)kz << 16), (uint32_t)vs | ((uint32_t)vz << 16));
    }
    __syncthreads();                       // every group has read the old length
    if (threadIdx.x == 0) {
        if (room) lens[0] = n_hi + 1;
        else report(status_word, ZIPVL_DEV_CAPACITY);
    }
}

// ---- decode over the two blocks ----------------------------------------------------------
// Eight adjacent lanes share a cached row of one KV head; a lane holds D/8 channels of the
// query heads that read that KV head (pre-scaled) and of their output accumulators.  With
// k^ = code * s_k + z_k the score is s_k * <q, code> + z_k * sum(q): the dot product runs on the
// integer codes (turned into floats by an OR into the mantissa of 2^23, no conversion
// instruction), and likewise o += (p * s_v) * code with p * z_v summed on the side.
// Split over the rows like decode_kernel; the chunk partials go to the same workspace layout
// and decode_merge_kernel finishes the step.
constexpr int kDqThreads = 128, kDqLanes = 8, kDqUnroll = 4;

__device__ __forceinline__ float code_to_float(uint32_t c) { return __uint_as_float(0x4B000000u | c) - 8388608.0f; }

template <bool kHalf, int D, int GT>
__global__ void __launch_bounds__(kDqThreads)
decode_quant_kernel(int Hq, int Hkv, float scale_log2, const unsigned short *__restrict__ q, QuantBlocks qb,
                    int32_t *lens, const zipvl_quant_cache *__restrict__ caches, int max_len, int chunk,
                    int n_chunks, float *__restrict__ ws, int *__restrict__ lens_ws, int32_t *status_word) {
    constexpr int CPL = D / kDqLanes;            // channels per lane: 16 or 8
    constexpr int RPW = 32 / kDqLanes;           // rows per warp per load: 4
    constexpr int NG = (kDqThreads / 32) * RPW;  // row groups per CTA: 16
    __shared__ float sm_o[NG][GT][D];
    __shared__ float sm_m[NG][GT], sm_l[NG][GT];
    grid_launch_dependents();
    grid_dependency_wait(q, lens, caches, qb.k_hi, qb.v_hi, qb.k_lo, qb.v_lo, qb.p_hi, qb.p_lo);
    const int b = blockIdx.z;                    // request
    const bool blocks_ok = request_blocks(caches, b, qb, lens);
    q += (long long)b * Hq * D;
    ws += (long long)b * Hq * n_chunks * (D + 2);
    lens_ws += 2 * b;
    const int G = Hq / Hkv;
    const int hkv = blockIdx.y, h0 = hkv * G;
    const int n_heads = min(GT, G);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rg = warp * RPW + lane / kDqLanes, lr = lane % kDqLanes;
    // the query slices of this lane and the sum of each (whole) query row
    float qv[GT][CPL], qsum[GT];
#pragma unroll
    for (int g = 0; g < GT; ++g) {
        float part = 0.f;
#pragma unroll
        for (int c0 = 0; c0 < CPL; c0 += 8) {
            float x[8];
            if (g < n_heads) unpack8s<kHalf>(*reinterpret_cast<const uint4 *>(q + (long long)(h0 + g) * D + lr * CPL + c0), x);
            else {
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) { qv[g][c0 + e] = x[e] * scale_log2; part += qv[g][c0 + e]; }
        }
#pragma unroll
        for (int o = kDqLanes / 2; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        qsum[g] = part;
    }
    int n_hi = blocks_ok ? lens[0] : 0, n_lo = blocks_ok ? lens[1] : 0;
    const bool bad = !blocks_ok || n_hi < 0 || n_lo < 0 || n_hi > qb.cap_hi || n_lo > qb.cap_lo;
    if (bad) {
        if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) report(status_word, ZIPVL_DEV_BAD_INDEX);
        n_hi = 0; n_lo = 0;
    }
    int total = n_hi + n_lo;
    if (total > max_len) {
        if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) report(status_word, ZIPVL_DEV_CAPACITY);
        total = max_len;
    }
    const int c0r = blockIdx.x * chunk;
    if (c0r < total) {
        const int c1r = min(total, c0r + chunk);
        float o[GT][CPL], zacc[GT], m[GT], l[GT];
#pragma unroll
        for (int g = 0; g < GT; ++g) {
            m[g] = -INFINITY; l[g] = 0.f; zacc[g] = 0.f;
#pragma unroll
            for (int c = 0; c < CPL; ++c) o[g][c] = 0.f;
        }
        for (int base = c0r; base < c1r; base += NG * kDqUnroll) {
            unsigned long long wk[kDqUnroll], wv[kDqUnroll];
            uint2 par[kDqUnroll];
            int bits[kDqUnroll];
            bool ok[kDqUnroll];
#pragma unroll
            for (int u = 0; u < kDqUnroll; ++u) {
                const int r = base + u * NG + rg;
                ok[u] = r < c1r;
                wk[u] = 0; wv[u] = 0; par[u] = make_uint2(0, 0); bits[u] = 4;
                if (ok[u]) {
                    const bool is_hi = r < n_hi;
                    const long long rh = (long long)(is_hi ? r : r - n_hi) * Hkv + hkv;
                    bits[u] = is_hi ? 4 : 2;
                    const int lane_bytes = CPL * bits[u] / 8;                 // 8, 4 (d 128) or 4, 2 (d 64)
                    const unsigned char *pk = (is_hi ? qb.k_hi : qb.k_lo) + rh * (D * bits[u] / 8) + lr * lane_bytes;
                    const unsigned char *pv = (is_hi ? qb.v_hi : qb.v_lo) + rh * (D * bits[u] / 8) + lr * lane_bytes;
                    if (lane_bytes == 8) {
                        wk[u] = *reinterpret_cast<const unsigned long long *>(pk);
                        wv[u] = *reinterpret_cast<const unsigned long long *>(pv);
                    } else if (lane_bytes == 4) {
                        wk[u] = *reinterpret_cast<const uint32_t *>(pk);
                        wv[u] = *reinterpret_cast<const uint32_t *>(pv);
                    } else {
                        wk[u] = *reinterpret_cast<const unsigned short *>(pk);
                        wv[u] = *reinterpret_cast<const unsigned short *>(pv);
                    }
                    par[u] = *reinterpret_cast<const uint2 *>((is_hi ? qb.p_hi : qb.p_lo) + rh * 4);
                }
            }
            float s[kDqUnroll][GT];
#pragma unroll
            for (int u = 0; u < kDqUnroll; ++u) {
                const uint32_t mask = (1u << bits[u]) - 1u;
                float dot[GT];
#pragma unroll
                for (int g = 0; g < GT; ++g) dot[g] = 0.f;
#pragma unroll
                for (int c = 0; c < CPL; ++c) {
                    const float cf = code_to_float((uint32_t)(wk[u] >> (bits[u] * c)) & mask);
#pragma unroll
                    for (int g = 0; g < GT; ++g) dot[g] = fmaf(qv[g][c], cf, dot[g]);
                }
                const float ks = storage_to_float<kHalf>((unsigned short)(par[u].x & 0xffffu));
                const float kz = storage_to_float<kHalf>((unsigned short)(par[u].x >> 16));
#pragma unroll
                for (int g = 0; g < GT; ++g) {
                    float dsum = dot[g];
#pragma unroll
                    for (int off = kDqLanes / 2; off > 0; off >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, off);
                    s[u][g] = ok[u] ? fmaf(ks, dsum, kz * qsum[g]) : -INFINITY;
                }
            }
#pragma unroll
            for (int g = 0; g < GT; ++g) {
                float mn = m[g];
#pragma unroll
                for (int u = 0; u < kDqUnroll; ++u) mn = fmaxf(mn, s[u][g]);
                if (mn == -INFINITY) continue;
                const float sc = fast_exp2(m[g] - mn);
                m[g] = mn;
                l[g] *= sc;
                zacc[g] *= sc;
#pragma unroll
                for (int c = 0; c < CPL; ++c) o[g][c] *= sc;
#pragma unroll
                for (int u = 0; u < kDqUnroll; ++u) s[u][g] = fast_exp2(s[u][g] - mn);
            }
#pragma unroll
            for (int u = 0; u < kDqUnroll; ++u) {
                const uint32_t mask = (1u << bits[u]) - 1u;
                const float vs = storage_to_float<kHalf>((unsigned short)(par[u].y & 0xffffu));
                const float vz = storage_to_float<kHalf>((unsigned short)(par[u].y >> 16));
                float w[GT];
#pragma unroll
                for (int g = 0; g < GT; ++g) {
                    const float p = (m[g] == -INFINITY) ? 0.f : s[u][g];
                    l[g] += p;
                    zacc[g] = fmaf(p, vz, zacc[g]);
                    w[g] = p * vs;
                }
#pragma unroll
                for (int c = 0; c < CPL; ++c) {
                    const float cf = code_to_float((uint32_t)(wv[u] >> (bits[u] * c)) & mask);
#pragma unroll
                    for (int g = 0; g < GT; ++g) o[g][c] = fmaf(w[g], cf, o[g][c]);
                }
            }
        }
        // combine the row groups of the CTA
#pragma unroll
        for (int g = 0; g < GT; ++g) {
#pragma unroll
            for (int c = 0; c < CPL; ++c) sm_o[rg][g][lr * CPL + c] = o[g][c] + zacc[g];
            if (lr == 0) { sm_m[rg][g] = m[g]; sm_l[rg][g] = l[g]; }
        }
        __syncthreads();
        for (int t = threadIdx.x; t < n_heads * D; t += kDqThreads) {
            const int g = t / D, c = t % D;
            float M = -INFINITY;
#pragma unroll
            for (int r = 0; r < NG; ++r) M = fmaxf(M, sm_m[r][g]);
            float Ls = 0.f, Os = 0.f;
#pragma unroll
            for (int r = 0; r < NG; ++r) {
                const float mr = sm_m[r][g];
                const float wgt = (mr == -INFINITY) ? 0.f : fast_exp2(mr - M);
                Ls += sm_l[r][g] * wgt;
                Os += sm_o[r][g][c] * wgt;
            }
            float *dst = ws + ((long long)(h0 + g) * n_chunks + blockIdx.x) * (D + 2);
            dst[2 + c] = Os;
            if (c == 0) { dst[0] = M; dst[1] = Ls; }
        }
    } else if ((int)threadIdx.x < n_heads) {
        float *dst = ws + ((long long)(h0 + threadIdx.x) * n_chunks + blockIdx.x) * (D + 2);
        dst[0] = -INFINITY;      // a chunk past the cache: an empty partial
        dst[1] = 0.f;
    }
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        lens_ws[0] = total;
        lens_ws[1] = 0;          // (the append kernel has already counted the new row)
    }
}

template <bool kHalf, int D>
zipvl_status run_quantize(const LayerArgs &a, const void *k, const void *v, const int32_t *idx,
                          const int32_t *k_dev, int k_max, const QuantBlocks &qb, int32_t *lens_out,
                          int32_t *status_word, cudaStream_t st) {
    const long long pairs = (long long)a.L * a.Hkv;
    const int per_cta = (kQuantThreads / 32) * (32 / (D / 8)) * kQuantIters;
    const long long grid = (pairs + per_cta - 1) / per_cta;
    const cudaError_t e = launch_dependent(quantize_kv_kernel<kHalf, D>, dim3((unsigned)grid), dim3(kQuantThreads), 0, st,
                                           a, (const unsigned short *)k, (const unsigned short *)v, idx, k_dev, k_max,
                                           qb, lens_out, status_word);
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "zipvl_quantize_kv: launch: %s", cudaGetErrorString(e));
    count_launches(1);
    return check_launch("zipvl_quantize_kv");
}

template <bool kHalf, int D>
zipvl_status run_decode_quant(const zipvl_decode_desc &d, float scale_log2, const void *q, const void *k_new,
                              const void *v_new, const QuantBlocks &qb, int32_t *lens,
                              const zipvl_quant_cache *caches, int max_len, void *out, void *ws,
                              int32_t *status_word, cudaStream_t st) {
    const int Hq = d.n_q_heads, Hkv = d.n_kv_heads, G = Hq / Hkv, B = d.batch;
    cudaError_t e = cudaSuccess;
    if (k_new) {
        e = launch_dependent(quant_append_kernel<kHalf, D>, dim3(B), dim3(Hkv * (D / 8)), 0, st, Hkv,
                             (const unsigned short *)k_new, (const unsigned short *)v_new, qb, lens, caches,
                             status_word);
        if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "zipvl_decode_quant: launch: %s", cudaGetErrorString(e));
        count_launches(1);
    }
    const int chunk = decode_chunk_rows(B, Hq, max_len);
    const int n_chunks = (max_len + chunk - 1) / chunk;
    float *wsf = reinterpret_cast<float *>(ws);
    int *lens_ws = reinterpret_cast<int *>(reinterpret_cast<char *>(ws) + decode_partial_bytes(B, Hq, D, max_len));
    const dim3 grid(n_chunks, Hkv, B);
#define ZIPVL_DQ(GT_)                                                                                       \
    e = launch_dependent(decode_quant_kernel<kHalf, D, GT_>, grid, dim3(kDqThreads), 0, st, Hq, Hkv, scale_log2, \
                         (const unsigned short *)q, qb, lens, caches, max_len, chunk, n_chunks, wsf,             \
                         lens_ws, status_word)
    if (G == 1) ZIPVL_DQ(1);
    else if (G == 2) ZIPVL_DQ(2);
    else ZIPVL_DQ(4);
#undef ZIPVL_DQ
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "zipvl_decode_quant: launch: %s", cudaGetErrorString(e));
    count_launches(1);
    // (the append kernel has counted the new rows: the merge writes no length; the words behind the
    // (length, appended) pairs stand in for its length array)
    return launch_decode_merge(d.dtype, D, Hq, B, chunk, n_chunks, wsf, lens_ws, lens_ws + 2 * B, out, st);
}

}  // namespace
}  // namespace zipvl

using namespace zipvl;

static zipvl_status check_blocks(const char *who, int Hkv, void *k_hi, void *v_hi, void *p_hi, int cap_hi, void *k_lo,
                                 void *v_lo, void *p_lo, int cap_lo, QuantBlocks *qb) {
    if (!k_hi || !v_hi || !p_hi || !k_lo || !v_lo || !p_lo) return fail(ZIPVL_ERR_INVALID_ARG, "%s: NULL cache block", who);
    if (cap_hi < 1 || cap_lo < 1) return fail(ZIPVL_ERR_INVALID_ARG, "%s: capacities %d / %d", who, cap_hi, cap_lo);
    if (((uintptr_t)k_hi | (uintptr_t)v_hi | (uintptr_t)p_hi | (uintptr_t)k_lo | (uintptr_t)v_lo | (uintptr_t)p_lo) & 15u)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: cache blocks must be 16-byte aligned", who);
    if (Hkv > 1024 / 16) return fail(ZIPVL_ERR_UNSUPPORTED, "%s: more than 64 KV heads", who);
    *qb = QuantBlocks{(unsigned char *)k_hi, (unsigned char *)v_hi, (unsigned char *)k_lo, (unsigned char *)v_lo,
                      (unsigned short *)p_hi, (unsigned short *)p_lo, cap_hi, cap_lo};
    return ZIPVL_OK;
}

extern "C" zipvl_status zipvl_quantize_kv(const zipvl_layer *l, const void *k, const void *v, const int32_t *idx,
                                          const int32_t *k_dev, int32_t k_max, void *k_hi, void *v_hi,
                                          void *params_hi, int32_t cap_hi, void *k_lo, void *v_lo,
                                          void *params_lo, int32_t cap_lo, int32_t *lens_out,
                                          int32_t *status_word, void *stream) {
    const char *who = "zipvl_quantize_kv";
    if (!l) return fail(ZIPVL_ERR_INVALID_ARG, "%s: layer is NULL", who);
    if (l->L < 1 || l->n_kv_heads < 1 || l->n_q_heads < 1 || l->n_q_heads % l->n_kv_heads)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: L %d heads %d / %d", who, l->L, l->n_q_heads, l->n_kv_heads);
    if ((l->dtype != ZIPVL_BF16 && l->dtype != ZIPVL_F16) || (l->head_dim != 64 && l->head_dim != 128))
        return fail(ZIPVL_ERR_UNSUPPORTED, "%s: dtype %d head_dim %d (16-bit storage, head_dim 64 or 128)", who,
                    l->dtype, l->head_dim);
    const long long ks = l->kv_stride_tok ? l->kv_stride_tok : (long long)l->n_kv_heads * l->head_dim;
    if (ks < (long long)l->n_kv_heads * l->head_dim || ks % 8)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: token stride %lld", who, ks);
    if (!k || !v || !idx || !k_dev || !lens_out) return fail(ZIPVL_ERR_INVALID_ARG, "%s: NULL pointer", who);
    if (k_max < 1 || k_max > l->L) return fail(ZIPVL_ERR_INVALID_ARG, "%s: k_max = %d not in [1, L]", who, k_max);
    if (((uintptr_t)k | (uintptr_t)v) & 15u) return fail(ZIPVL_ERR_INVALID_ARG, "%s: k, v must be 16-byte aligned", who);
    QuantBlocks qb;
    const zipvl_status s = check_blocks(who, l->n_kv_heads, k_hi, v_hi, params_hi, cap_hi, k_lo, v_lo, params_lo, cap_lo, &qb);
    if (s != ZIPVL_OK) return s;
    LayerArgs a{};
    a.L = l->L; a.Hq = l->n_q_heads; a.Hkv = l->n_kv_heads; a.D = l->head_dim; a.G = a.Hq / a.Hkv;
    a.kv_stride = ks; a.q_stride = (long long)a.Hq * a.D; a.half = (l->dtype == ZIPVL_F16); a.n_seq = 1;
    cudaStream_t st = (cudaStream_t)stream;
    if (a.half) return a.D == 128 ? run_quantize<true, 128>(a, k, v, idx, k_dev, k_max, qb, lens_out, status_word, st)
                                  : run_quantize<true, 64>(a, k, v, idx, k_dev, k_max, qb, lens_out, status_word, st);
    return a.D == 128 ? run_quantize<false, 128>(a, k, v, idx, k_dev, k_max, qb, lens_out, status_word, st)
                      : run_quantize<false, 64>(a, k, v, idx, k_dev, k_max, qb, lens_out, status_word, st);
}

// what the two decode entries check alike
static zipvl_status check_decode_quant(const char *who, const zipvl_decode_desc *d, const void *q, const void *k_new,
                                       const void *v_new, int max_len, const void *out, const void *ws) {
    if (!d) return fail(ZIPVL_ERR_INVALID_ARG, "%s: desc is NULL", who);
    if (d->n_q_heads < 1 || d->n_kv_heads < 1 || d->n_q_heads % d->n_kv_heads)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: heads %d / %d", who, d->n_q_heads, d->n_kv_heads);
    const int G = d->n_q_heads / d->n_kv_heads;
    if ((d->dtype != ZIPVL_BF16 && d->dtype != ZIPVL_F16) || (d->head_dim != 64 && d->head_dim != 128) ||
        (G != 1 && G != 2 && G != 4))
        return fail(ZIPVL_ERR_UNSUPPORTED, "%s: dtype %d head_dim %d group %d (16-bit storage, head_dim 64 or 128, "
                    "1, 2 or 4 query heads per KV head)", who, d->dtype, d->head_dim, G);
    if (!q || !out || !ws) return fail(ZIPVL_ERR_INVALID_ARG, "%s: NULL pointer", who);
    if ((k_new == NULL) != (v_new == NULL))
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: k_new and v_new must both be given or both NULL", who);
    if (max_len < 1) return fail(ZIPVL_ERR_INVALID_ARG, "%s: max_len = %d", who, max_len);
    if (!(d->softmax_scale >= 0.f) || isinf(d->softmax_scale)) return fail(ZIPVL_ERR_INVALID_ARG, "%s: softmax_scale", who);
    if (((uintptr_t)q | (uintptr_t)out | (uintptr_t)ws | (uintptr_t)k_new | (uintptr_t)v_new) & 15u)
        return fail(ZIPVL_ERR_INVALID_ARG, "%s: tensors must be 16-byte aligned", who);
    return ZIPVL_OK;
}

static zipvl_status dispatch_decode_quant(const zipvl_decode_desc &d, float scale, const void *q, const void *k_new,
                                          const void *v_new, const QuantBlocks &qb, int32_t *lens,
                                          const zipvl_quant_cache *caches, int max_len, void *out, void *ws,
                                          int32_t *status_word, cudaStream_t st) {
    const bool half = d.dtype == ZIPVL_F16;
    if (half) return d.head_dim == 128 ? run_decode_quant<true, 128>(d, scale, q, k_new, v_new, qb, lens, caches, max_len, out, ws, status_word, st)
                                       : run_decode_quant<true, 64>(d, scale, q, k_new, v_new, qb, lens, caches, max_len, out, ws, status_word, st);
    return d.head_dim == 128 ? run_decode_quant<false, 128>(d, scale, q, k_new, v_new, qb, lens, caches, max_len, out, ws, status_word, st)
                             : run_decode_quant<false, 64>(d, scale, q, k_new, v_new, qb, lens, caches, max_len, out, ws, status_word, st);
}

extern "C" zipvl_status zipvl_decode_quant(const zipvl_decode_desc *d, const void *q, const void *k_new,
                                           const void *v_new, void *k_hi, void *v_hi, void *params_hi,
                                           int32_t cap_hi, void *k_lo, void *v_lo, void *params_lo,
                                           int32_t cap_lo, int32_t *lens, int32_t max_len, void *out, void *ws,
                                           size_t ws_bytes, int32_t *status_word, void *stream) {
    const char *who = "zipvl_decode_quant";
    const zipvl_status sv = check_decode_quant(who, d, q, k_new, v_new, max_len, out, ws);
    if (sv != ZIPVL_OK) return sv;
    if (d->batch != 1) return fail(ZIPVL_ERR_UNSUPPORTED, "%s: batch %d (one request per call)", who, d->batch);
    if (!lens) return fail(ZIPVL_ERR_INVALID_ARG, "%s: NULL pointer", who);
    QuantBlocks qb;
    const zipvl_status s = check_blocks(who, d->n_kv_heads, k_hi, v_hi, params_hi, cap_hi, k_lo, v_lo, params_lo, cap_lo, &qb);
    if (s != ZIPVL_OK) return s;
    const size_t need = (decode_ws_bytes(1, d->n_q_heads, d->head_dim, max_len) + 255) & ~(size_t)255;
    if (ws_bytes < need) return fail(ZIPVL_ERR_WORKSPACE, "%s: workspace %zu < %zu", who, ws_bytes, need);
    const float scale = (d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / sqrtf((float)d->head_dim)) * kLog2e;
    return dispatch_decode_quant(*d, scale, q, k_new, v_new, qb, lens, nullptr, max_len, out, ws, status_word,
                                 (cudaStream_t)stream);
}

extern "C" zipvl_status zipvl_decode_quant_batch(const zipvl_decode_desc *d, const void *q, const void *k_new,
                                                 const void *v_new, const zipvl_quant_cache *caches,
                                                 int32_t max_len, void *out, void *ws, size_t ws_bytes,
                                                 int32_t *status_word, void *stream) {
    const char *who = "zipvl_decode_quant_batch";
    const zipvl_status s = check_decode_quant(who, d, q, k_new, v_new, max_len, out, ws);
    if (s != ZIPVL_OK) return s;
    if (d->batch < 1 || d->batch > 65535) return fail(ZIPVL_ERR_INVALID_ARG, "%s: batch %d not in [1, 65535]", who, d->batch);
    if (d->n_kv_heads > 1024 / 16) return fail(ZIPVL_ERR_UNSUPPORTED, "%s: more than 64 KV heads", who);
    if (!caches || ((uintptr_t)caches & 7u)) return fail(ZIPVL_ERR_INVALID_ARG, "%s: caches is NULL or misaligned", who);
    const size_t need = (decode_ws_bytes(d->batch, d->n_q_heads, d->head_dim, max_len) + 255) & ~(size_t)255;
    if (ws_bytes < need) return fail(ZIPVL_ERR_WORKSPACE, "%s: workspace %zu < %zu", who, ws_bytes, need);
    const float scale = (d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / sqrtf((float)d->head_dim)) * kLog2e;
    return dispatch_decode_quant(*d, scale, q, k_new, v_new, QuantBlocks{}, nullptr, caches, max_len, out, ws, status_word,
                                 (cudaStream_t)stream);
}
