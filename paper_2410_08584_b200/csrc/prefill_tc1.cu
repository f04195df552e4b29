// Sparse causal prefill attention, one 128-row query tile per CTA, two CTAs per SM
// (Algorithm 1: attention over Q[T], K[T], V[T]; Eq. 2 on the gathered tokens).
// The kernel for short and medium kept sets (a few thousand tokens), where the launch
// is a few waves of unequal work items: items of 128 query rows are half as long as the
// 256-row items of prefill_tc.cu, their ragged last item costs one 128-row diagonal, and
// the second CTA on the SM fills the time a CTA spends in its prologue (index -> row
// gather -> first MMA), in its epilogue, and waiting on its own softmax -> MMA chain.
//
// CTA = (query head, tile of 128 gathered query rows); key / value tiles of 128 gathered
// tokens up to the diagonal.  256 threads:
//   warps 0-3  softmax (thread = query row = TMEM lane): exact tile maximum, then
//              P = exp2(S*scale - m) written back over S in the storage type; the running
//              maximum moves only when a tile outgrows it by 2^32 (2^8 for IEEE half);
//              at the end O / l goes out through the query buffer as whole 256-byte rows.
//   warp 4     issues tcgen05.mma: S = Q K(n)^T (shared-memory operands), then, when P(n)
//              is in tensor memory, O += P(n) V(n) and at once S = Q K(n+1)^T.
//   warps 5-6  producers: the index list drives the loads.  Sixteen lanes copy one
//              gathered 256-byte row with 16-byte async copies straight into the
//              128-byte-swizzled layout the tensor core reads.  One K and one V buffer:
//              K(n+1) is fetched while softmax(n) runs, V(n+1) once PV(n) has read V(n).
//   warp 7     zeroes the rows of dropped tokens (PADDED output) while the attention runs
//              and, in the fused call, copies the CTA's own 128 K and V rows (its diagonal
//              tile, already in shared memory) to the compacted cache.
// Tensor memory: 256 columns (S | O, 128 fp32 columns each; P aliases the front of S), so
// two CTAs share an SM's 512.  Shared memory: Q, K, V tiles of 32 KB.  Every wait is
// bounded; a wait that runs out sets ZIPVL_DEV_TIMEOUT and all roles unwind to the exit.
#include <type_traits>

#include "tc.cuh"
#include "tc_ptx.cuh"

namespace zipvl {
namespace {

using namespace ptx;

constexpr int kD = 128;               // head_dim
constexpr int kBM = 128, kBN = 128;   // query / key tile
constexpr int kHalfBytes = 128 * 128;        // 128 rows x 64 elements (one swizzle atom wide)
constexpr int kTileBytes = 2 * kHalfBytes;   // 128 rows x 128 elements
constexpr int kThreads1 = 256;        // two warpgroups: softmax | issuer, producers, helper
constexpr int kRegsSoftmax = 200, kRegsOther = 56;
constexpr uint32_t kTmemCols1 = 256;
constexpr float kRescaleThreshold = 32.0f, kRescaleThresholdHalf = 8.0f;

struct Barriers1 {
    uint64_t q_full;      // 128 softmax threads: their query rows are in shared memory
    uint64_t k_full;      // 64 producer lanes: K(n) has landed           (phase n)
    uint64_t v_full;      // 64 producer lanes: V(n) has landed           (phase n)
    uint64_t s_full;      // commit behind QK(n): S(n) is in tensor memory, the K buffer is free
    uint64_t p_full;      // 128 softmax threads: P(n) is in tensor memory
    uint64_t pv_done;     // commit behind PV(n): the V buffer is free, O holds tiles 0..n
    uint64_t o_done;      // commit behind the last PV
    uint64_t tail_full;   // the issuer saw K and V of the diagonal tile land
    uint32_t tmem_base;
    int abort_flag;
};

constexpr size_t kSmemBytes1 = 3 * kTileBytes + sizeof(Barriers1) + 1024;

// Gather 32 rows of 256 bytes into a swizzled tile with one warp.  Lane l holds the token of
// row (row0 + l) in my_tok (-1 = zero-fill); row0 is a multiple of 32 and the tile is
// 1024-byte aligned.  Sixteen adjacent lanes copy one row (16 chunks of 16 B): lanes 0-15 row
// i, lanes 16-31 row i + 16.
template <bool kAllValid>
__device__ __forceinline__ void gather_rows32_impl(uint32_t tile, int row0, int my_tok,
                                                   const __nv_bfloat16 *base, unsigned int stride_bytes,
                                                   int lane) {
    const int c = lane & 15, sub = lane >> 4;
    const char *src_lane = reinterpret_cast<const char *>(base) + c * 16;
    const uint32_t dst_lane = (tile + (row0 + 16 * sub) * 128 + (c >> 3) * kHalfBytes) | ((c & 7) << 4);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int t = __shfl_sync(0xffffffffu, my_tok, i, 16);        // row i of my half-warp
        const uint32_t dst = (dst_lane ^ ((i & 7) << 4)) + i * 128;
        if (kAllValid)
            cp_async16(dst, src_lane + (unsigned long long)(unsigned int)t * stride_bytes, 16u);
        else
            cp_async16(dst, src_lane + (unsigned long long)(unsigned int)(t < 0 ? 0 : t) * stride_bytes,
                       t >= 0 ? 16u : 0u);
    }
}
__device__ __forceinline__ void gather_rows32(uint32_t tile, int row0, int my_tok,
                                              const __nv_bfloat16 *base, long long stride, int lane) {
    const unsigned int stride_bytes = (unsigned int)(stride * 2);     // (checked by the host: < 2^31)
    if (__all_sync(0xffffffffu, my_tok >= 0)) gather_rows32_impl<true>(tile, row0, my_tok, base, stride_bytes, lane);
    else gather_rows32_impl<false>(tile, row0, my_tok, base, stride_bytes, lane);
}

template <bool kHalf>
__global__ void __launch_bounds__(kThreads1, 2)
prefill_tc1_kernel(LayerArgs a, const __nv_bfloat16 *__restrict__ q,
                   const __nv_bfloat16 *__restrict__ k, const __nv_bfloat16 *__restrict__ v,
                   const int32_t *__restrict__ idx, const int32_t *__restrict__ k_dev, int k_max,
                   __nv_bfloat16 *__restrict__ out, int out_mode, __nv_bfloat16 *__restrict__ kc,
                   __nv_bfloat16 *__restrict__ vc, int capacity, int32_t *__restrict__ len_out,
                   int32_t *status_word) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char *gen = smem_raw + (base - raw);
    const uint32_t sQ = base, sK = base + kTileBytes, sV = base + 2 * kTileBytes;
    Barriers1 *bar = reinterpret_cast<Barriers1 *>(gen + 3 * kTileBytes);
    volatile int *abort_flag = &bar->abort_flag;

    // set-up that needs no global memory first: it overlaps the previous kernel's drain
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_launch_dependents();
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar->q_full), 128);
        mbar_init(smem_u32(&bar->k_full), 64);
        mbar_init(smem_u32(&bar->v_full), 64);
        mbar_init(smem_u32(&bar->s_full), 1);
        mbar_init(smem_u32(&bar->p_full), 128);
        mbar_init(smem_u32(&bar->pv_done), 1);
        mbar_init(smem_u32(&bar->o_done), 1);
        mbar_init(smem_u32(&bar->tail_full), 1);
        bar->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 4) tmem_alloc(smem_u32(&bar->tmem_base), kTmemCols1);
    grid_dependency_wait(q, k, v, idx, k_dev);   // k_dev and idx are the previous kernel's output
    int n_valid = *k_dev;
    if (n_valid > k_max || n_valid < 0) {
        if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0)
            report(status_word, ZIPVL_DEV_CAPACITY);
        n_valid = n_valid < 0 ? 0 : k_max;
    }
    // blocks are dispatched x-fastest: x = head, y = tile, so every head of the longest
    // diagonal starts first (longest-processing-time order); tiles past the actual k map to
    // the last rows of the grid and return at once
    const int n_qt = (n_valid + kBM - 1) / kBM;
    const int qt = n_qt - 1 - (int)blockIdx.y;
    const int q0 = qt * kBM;
    const bool no_work = (qt < 0 || (int)blockIdx.x >= a.Hq);
    const int h = blockIdx.x, g = h / a.G;
    const int n_kv = qt + 1;                        // key tiles 0 .. qt (the diagonal)

    auto token_of = [&](int i) {
        if (i >= n_valid) return -1;
        int t = idx[i];
        if (t < 0 || t >= a.L) { report(status_word, ZIPVL_DEV_BAD_INDEX); t = -1; }
        return t;
    };
    // the first token index a loading thread needs is fetched before the set-up barrier
    int first_tok = -1;
    if (!no_work) {
        if (warp < 4) first_tok = token_of(q0 + warp * 32 + lane);
        else if (warp == 5 || warp == 6) first_tok = token_of((warp - 5) * 64 + lane);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bar->tmem_base;
    if (no_work) {
        if (warp == 4) tmem_dealloc(tmem, kTmemCols1);
        if (n_valid == 0 && blockIdx.y == 0 && (int)blockIdx.x < a.Hq) {
            // nothing kept: an all-zero PADDED output and a cache of length 0
            if (out_mode == ZIPVL_OUT_PADDED) {
                const uint4 z = make_uint4(0, 0, 0, 0);
                for (int e = threadIdx.x; e < a.L * 16; e += kThreads1)
                    reinterpret_cast<uint4 *>(out + ((long long)(e >> 4) * a.Hq + h) * kD)[e & 15] = z;
            }
            if (kc != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *len_out = 0;
        }
        return;
    }

    if (warp >= 4) {
        reg_dec<kRegsOther>();
        if (warp == 5 || warp == 6) {
            // ------------------------------ producers ------------------------------
            // Load sequence K0 V0 K1 V1 ...  K(n) may overwrite the K buffer once QK(n-1) is
            // done (s_full, phase n-1), V(n) the V buffer once PV(n-1) is (pv_done, phase n-1):
            // the same order in which those events happen.  A load is issued as soon as its
            // buffer is free, up to two in flight; the thread blocks on a buffer only when it
            // has nothing in flight, so a landed tile is never announced late.
            const int rows0 = (warp - 5) * 64;      // this warp's 64 rows of every 128-row tile
            const int total = 2 * n_kv;
            int tok0 = first_tok, tok1 = -1;
            auto issue = [&](int seq) {
                const int n = seq >> 1;
                if ((seq & 1) == 0) {
                    if (seq > 0) tok0 = token_of(n * kBN + rows0 + lane);
                    tok1 = token_of(n * kBN + rows0 + 32 + lane);
                }
                const __nv_bfloat16 *src = ((seq & 1) ? v : k) + (long long)g * kD;
                const uint32_t dst = (seq & 1) ? sV : sK;
                gather_rows32(dst, rows0, tok0, src, a.kv_stride, lane);
                gather_rows32(dst, rows0 + 32, tok1, src, a.kv_stride, lane);
                cp_async_commit();
            };
            auto buffer_free = [&](int seq, bool block) {
                const int n = seq >> 1;
                if (n == 0) return true;
                const uint32_t b = smem_u32((seq & 1) ? &bar->pv_done : &bar->s_full);
                const uint32_t par = (n - 1) & 1;
                if (block) { mbar_wait(b, par, abort_flag); return true; }
                return warp_try_wait(b, par);
            };
            int issued = 0;
            for (int seq = 0; seq < total; ++seq) {
                while (issued < total && issued - seq < 2 && buffer_free(issued, issued == seq))
                    issue(issued++);
                if (issued - 1 - seq >= 1) cp_async_wait<1>();
                else cp_async_wait<0>();
                fence_proxy_async();
                mbar_arrive(smem_u32((seq & 1) ? &bar->v_full : &bar->k_full));
            }
        } else if (warp == 7) {
            // ---------------- zero-fill of dropped tokens' rows, fused KV compaction ----------------
            if (out_mode == ZIPVL_OUT_PADDED) {
                const uint4 z = make_uint4(0, 0, 0, 0);
                const int sub = lane >> 4, ch = lane & 15;
                auto clear_rows = [&](int r0, int r1) {
                    for (int zr = r0 + sub; zr < r1; zr += 2)
                        reinterpret_cast<uint4 *>(out + ((long long)zr * a.Hq + h) * kD)[ch] = z;
                };
                for (int i0 = 0; i0 < kBM; i0 += 32) {
                    const int i = q0 + i0 + lane;
                    const int t = token_of(i);
                    int lo = 0, hi = 0;                       // my gap: rows [lo, hi)
                    if (t >= 0) {
                        // a previous entry that is out of range, or not below this one (the
                        // list must ascend), is read as "no gap": nothing is cleared for it
                        const int tp = (i == 0) ? -1 : idx[i - 1];
                        lo = (i == 0) ? 0 : ((tp >= 0 && tp < t) ? tp + 1 : t);
                        hi = t;
                    }
                    const bool last = (t >= 0 && i == n_valid - 1);
                    unsigned int gaps = __ballot_sync(0xffffffffu, hi > lo);
                    const unsigned int tail = __ballot_sync(0xffffffffu, last);
                    while (gaps) {
                        const int src = __ffs(gaps) - 1;
                        gaps &= gaps - 1;
                        clear_rows(__shfl_sync(0xffffffffu, lo, src), __shfl_sync(0xffffffffu, hi, src));
                    }
                    if (tail) {
                        const int src = __ffs(tail) - 1;
                        clear_rows(__shfl_sync(0xffffffffu, t, src) + 1, a.L);
                    }
                }
            }
            // Fused KV compaction (Algorithm 1: K = K[T], V = V[T]).  The diagonal key tile of
            // this CTA holds exactly the K and V rows of its own 128 kept tokens, gathered into
            // shared memory for the attention and never overwritten (they are the last loads).
            // The CTA of the first query head of a KV group writes them out from there.
            if (kc != nullptr && h % a.G == 0) {
                const int lim = min(n_valid, capacity);
                const int sub = lane >> 4, ch = lane & 15;
                mbar_wait(smem_u32(&bar->tail_full), 0, abort_flag);
                for (int kind = 0; kind < 2; ++kind) {
                    const unsigned char *tile = gen + (size_t)kTileBytes * (1 + kind);
                    __nv_bfloat16 *dstc = kind ? vc : kc;
#pragma unroll 4
                    for (int r = sub; r < kBN; r += 2) {
                        const int i = q0 + r;
                        if (i >= lim) continue;    // (a row with an invalid index is all zeros here)
                        const uint4 w = *reinterpret_cast<const uint4 *>(
                            tile + (ch >> 3) * kHalfBytes + r * 128 + (((ch & 7) ^ (r & 7)) << 4));
                        reinterpret_cast<uint4 *>(dstc + ((long long)i * a.Hkv + g) * kD)[ch] = w;
                    }
                }
                if (blockIdx.x == 0 && blockIdx.y == 0 && lane == 0) {
                    *len_out = lim;
                    if (n_valid > capacity) report(status_word, ZIPVL_DEV_CAPACITY);
                }
            }
        } else {
            // ------------------------------ MMA issuer (warp 4) ------------------------------
            // the whole warp runs the (warp-uniform) control flow; one elected lane issues
            const bool leader = elect_one();
            constexpr uint32_t idesc_qk = idesc_f16kind(kBM, kBN, false, false, !kHalf);
            constexpr uint32_t idesc_pv = idesc_f16kind(kBM, kD, false, true, !kHalf);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t lo_q = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t lo_k = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t lo_v = ((sV & 0x3FFFFu) >> 4) | ((uint32_t)(kHalfBytes >> 4) << 16);
            auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
            auto qk = [&]() {                          // S = Q K^T
                if (leader) {
#pragma unroll
                    for (int kb = 0; kb < kD / 16; ++kb) {
                        const uint32_t o = ((kb >> 2) * kHalfBytes + (kb & 3) * 32) >> 4;
                        mma_ss(tmem, desc(lo_q + o), desc(lo_k + o), idesc_qk, kb > 0);
                    }
                    mma_commit(smem_u32(&bar->s_full));
                }
                __syncwarp();
            };
            auto pv = [&](int n) {                     // O += P V: P from tensor memory, V MN-major
                if (leader) {
#pragma unroll
                    for (int kb = 0; kb < kBN / 16; ++kb)
                        mma_ts(tmem + 128, tmem + kb * 8, desc(lo_v + kb * (2048 >> 4)), idesc_pv,
                               (n > 0 || kb > 0));
                }
                __syncwarp();
            };
            mbar_wait(smem_u32(&bar->q_full), 0, abort_flag);
            mbar_wait(smem_u32(&bar->k_full), 0, abort_flag);
            tc_fence_after();
            if (!*abort_flag) qk();
            for (int n = 0; n < n_kv && !*abort_flag; ++n) {
                const bool more = (n + 1 < n_kv);
                // the loads this step reads are waited for while the softmax works, so a
                // finished P finds the way to the tensor pipe clear
                mbar_wait(smem_u32(&bar->v_full), n & 1, abort_flag);
                if (more) mbar_wait(smem_u32(&bar->k_full), (n + 1) & 1, abort_flag);
                else if (leader) mbar_arrive(smem_u32(&bar->tail_full));   // K and V of the diagonal are in
                mbar_wait(smem_u32(&bar->p_full), n & 1, abort_flag);
                tc_fence_after();
                if (*abort_flag) break;
                pv(n);
                if (more) {
                    if (leader) mma_commit(smem_u32(&bar->pv_done));
                    qk();
                } else if (leader) {
                    mma_commit(smem_u32(&bar->o_done));
                }
            }
        }
    } else {
        // --------------------------- softmax / epilogue ---------------------------
        reg_inc<kRegsSoftmax>();
        const int row = threadIdx.x;                    // TMEM lane, query row in tile
        gather_rows32(sQ, warp * 32, first_tok, q + (long long)h * kD, a.q_stride, lane);
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        mbar_arrive(smem_u32(&bar->q_full));
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        const uint32_t tS = lane_base;
        const uint32_t tO = lane_base + 128;
        float m = -INFINITY, l = 0.f;
        const uint64_t scale2 = pack2f(a.scale_log2, a.scale_log2);
        const int quad = warp;                          // this warp's 32-row (and, on the diagonal, 32-column) block
        auto tile = [&](auto diag_c, int n) {
            constexpr bool kDiag = decltype(diag_c)::value;
            uint32_t sr[4][32];
            tmem_ld32(tS, sr[0]);
            tmem_ld32(tS + 32, sr[1]);
            tmem_wait_ld();
            tmem_ld32(tS + 64, sr[2]);      // lands while the first half is scanned
            tmem_ld32(tS + 96, sr[3]);
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            // On the diagonal tile row r sees columns 0..r.  A warp's 32 rows share their
            // 32-column chunk: chunks below it are fully visible, the chunk with the warp's
            // own index is cut per lane (column e <= lane), chunks above it are fully masked.
            auto scan = [&](int c) {
                if (kDiag && c > quad) return;
                const bool cut = kDiag && c == quad;
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float v0 = __uint_as_float(sr[c][e]), v1 = __uint_as_float(sr[c][e + 1]);
                    if (cut) {
                        if (e > lane) v0 = -INFINITY;
                        if (e + 1 > lane) v1 = -INFINITY;
                    }
                    mx4[(e >> 1) & 3] = max3(mx4[(e >> 1) & 3], v0, v1);
                }
            };
            scan(0);
            scan(1);
            tmem_wait_ld();
            scan(2);
            scan(3);
            const float m_tile = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;
            float alpha = 1.f;
            const bool grow = (m_tile > m + (kHalf ? kRescaleThresholdHalf : kRescaleThreshold));   // always true on the first tile
            if (grow) {
                alpha = ex2(m - m_tile);
                m = m_tile;
            }
            const bool rescale = __any_sync(0xffffffffu, grow) && n > 0;
            const uint64_t neg_m2 = pack2f(-m, -m);
            uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t p16[16];
                if (kDiag && c > quad) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) p16[e] = 0u;       // fully masked: no exponentials
                } else {
                    const bool cut = kDiag && c == quad;
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const uint64_t x2 = fma2(pack2u(sr[c][e], sr[c][e + 1]), scale2, neg_m2);
                        float x0, x1;
                        unpack2f(x2, x0, x1);
                        float p0 = ex2(x0), p1 = ex2(x1);
                        if (cut) {
                            if (e > lane) p0 = 0.f;
                            if (e + 1 > lane) p1 = 0.f;
                        }
                        sum2[(e >> 1) & 3] = add2(sum2[(e >> 1) & 3], pack2f(p0, p1));
                        p16[e >> 1] = pack16<kHalf>(p0, p1);
                    }
                }
                tmem_st16(tS + c * 16, p16);   // P overwrites the front of S: every S column is in registers
            }
            float sa, sb, sc, sd;
            unpack2f(add2(sum2[0], sum2[1]), sa, sb);
            unpack2f(add2(sum2[2], sum2[3]), sc, sd);
            l = l * alpha + ((sa + sb) + (sc + sd));
            if (rescale) {
                // O is complete through tile n-1: the commit that announced S(n) was issued
                // after PV(n-1) and covers it
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tO + c * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                    tmem_st32(tO + c * 32, r);
                }
            }
            tmem_wait_st();
        };
        for (int n = 0; n < n_kv; ++n) {
            mbar_wait(smem_u32(&bar->s_full), n & 1, abort_flag);
            tc_fence_after();
            if (n == qt) tile(std::true_type{}, n);
            else tile(std::false_type{}, n);
            tc_fence_before();
            mbar_arrive(smem_u32(&bar->p_full));
        }
        // ---- epilogue: O / l -> storage type -> global ----
        mbar_wait(smem_u32(&bar->o_done), 0, abort_flag);
        tc_fence_after();
        const int i = q0 + row;
        const int t = first_tok;
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const bool padded = (out_mode == ZIPVL_OUT_PADDED);
        __nv_bfloat16 *dst = nullptr;
        if (t >= 0 && !*abort_flag)
            dst = out + ((long long)(padded ? t : i) * a.Hq + h) * kD;
        // through the query buffer (no MMA reads it any more): each warp stages its own 32
        // rows, 16-byte chunks XOR-swizzled by the row, then writes whole 256-byte rows
        unsigned char *stage = gen + (size_t)warp * (32 * 256);
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(tO + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
                uint4 w;
                w.x = pack16<kHalf>(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
                w.y = pack16<kHalf>(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
                w.z = pack16<kHalf>(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
                w.w = pack16<kHalf>(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
                const int chunk = c * 4 + (e >> 3);
                *reinterpret_cast<uint4 *>(stage + lane * 256 + ((chunk ^ (lane & 15)) << 4)) = w;
            }
        }
        __syncwarp();
        {
            const int sub = lane >> 4, ch = lane & 15;
#pragma unroll 4
            for (int rr = sub; rr < 32; rr += 2) {
                const unsigned long long d = __shfl_sync(0xffffffffu, (unsigned long long)dst, rr);
                const uint4 w = *reinterpret_cast<const uint4 *>(stage + rr * 256 + ((ch ^ (rr & 15)) << 4));
                if (d) reinterpret_cast<uint4 *>(d)[ch] = w;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(status_word, ZIPVL_DEV_TIMEOUT);
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols1);
    }
}

}  // namespace

zipvl_status launch_prefill_tc1(const LayerArgs &a, const void *q, const void *k, const void *v,
                                const int32_t *idx, const int32_t *k_dev, int k_max, void *out,
                                int out_mode, void *k_cache, void *v_cache, int capacity,
                                int32_t *len_out, int32_t *status_word, cudaStream_t st) {
    auto kernel = a.half ? prefill_tc1_kernel<true> : prefill_tc1_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes1);
    if (e != cudaSuccess)
        return fail(ZIPVL_ERR_CUDA, "sparse_prefill: smem opt-in: %s", cudaGetErrorString(e));
    dim3 grid(a.Hq, (k_max + kBM - 1) / kBM);
    e = launch_dependent(kernel, grid, dim3(kThreads1), kSmemBytes1, st, a, (const __nv_bfloat16 *)q,
                         (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, idx, k_dev, k_max,
                         (__nv_bfloat16 *)out, out_mode, (__nv_bfloat16 *)k_cache,
                         (__nv_bfloat16 *)v_cache, capacity, len_out, status_word);
    if (e != cudaSuccess)
        return fail(ZIPVL_ERR_CUDA, "sparse_prefill: launch: %s", cudaGetErrorString(e));
    count_launches(1);
    return check_launch("zipvl_sparse_prefill");
}

}  // namespace zipvl
