// Probe scoring on the tensor cores (supplementary Eq. A with the causal mask of
// Eq. 2; column sums of Eq. 6; normalisation of Eq. 8).  bf16 or fp16, head_dim 64, 96 or
// 128, up to 128 probe rows.
//
// A column sum of a row-softmax needs each row's final max and denominator, so
// the probe x key contraction runs twice; the attention matrix only ever exists
// as 128 x 128 fp32 tiles in tensor memory.
//   stats   S  = Q' K^T   (M = probes, N = keys): one thread per probe row keeps
//           a running (max, sum) over the key tiles of its chunk;
//   colsum  S^T = K Q'^T  (M = keys, N = probes): the SAME two shared-memory
//           tiles with the operand roles swapped, so one thread owns one key
//           and sums exp2(s - m_r) / l_r over the probes that see it.
// CTA = (query head, chunk of key tiles).  The 128 gathered probe rows of the
// head stay resident in shared memory; key tiles stream in through TMA (tensor
// map over K as [L, Hkv*d], 128-byte swizzle, two 64-column boxes per tile) into
// a two-deep ring; one thread issues tcgen05.mma into one of two TMEM buffers so
// the next tile's MMA overlaps the current tile's exponentials.
// Every head adds its column sums to 64-bit fixed-point totals (integer adds: no order to
// depend on, so results repeat bit for bit); the last CTA to finish a key chunk turns the
// totals into floats and normalises.
#include <cuda.h>

#include "tc.cuh"
#include "tc_ptx.cuh"

namespace zipvl {
namespace {

using namespace ptx;

// The shared-memory tiles are 128 columns wide (two 64-column swizzle atoms); head_dim 64 and 96 use
// the front of them -- fewer 16-byte chunks per gathered row, fewer k-blocks per MMA
constexpr int kTile = 128, kMaxProbe = 128;
constexpr int kHalfBytes = 128 * 128;
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kKStages = 2;
constexpr int kThreadsSc = 192;
constexpr float kFxScale = 1099511627776.0f;   // 2^40: units of the fixed-point column totals
constexpr uint32_t kTmemColsSc = 256;

struct ScBarriers {
    uint64_t q_full;
    uint64_t k_full[kKStages];
    uint64_t k_empty[kKStages];
    uint64_t s_full[2];
    uint64_t s_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

constexpr size_t kScSmem = kTileBytes * (1 + kKStages) + 3 * kMaxProbe * 4 + sizeof(ScBarriers) + 1024;

template <int n_chunks16>
__device__ __forceinline__ void gather_row_sw128(uint32_t tile, int row, const __nv_bfloat16 *src,
                                                 bool valid) {
    const uint32_t bytes = valid ? 16u : 0u;
    const uint32_t rbase = tile + row * 128;
    const int sw = row & 7;
#pragma unroll
    for (int c = 0; c < 16; ++c)
        if (c < n_chunks16)
            cp_async16(rbase + (c >> 3) * kHalfBytes + (((c & 7) ^ sw) << 4), src + c * 8, bytes);
}

// MODE 0: row statistics.  MODE 1: column sums.
// barrier over the 128 consumer threads only (named barrier 1)
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// kHd: head_dim (64, 96 or 128) as a compile-time constant
template <int MODE, int kHd>
__global__ void __launch_bounds__(kThreadsSc, 2)   // two CTAs per SM hide each other's latency
score_tc_kernel(const __grid_constant__ CUtensorMap kmap, LayerArgs a,
                const __nv_bfloat16 *__restrict__ q, const int32_t *__restrict__ probe_pos, int P,
                int tiles_per_chunk, int n_chunks, float2 *__restrict__ stats,
                unsigned long long *__restrict__ accfx, int *__restrict__ counters,
                float *__restrict__ acc, float *__restrict__ norm, int32_t *status_word) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char *gen = smem_raw + (base - raw);
    const uint32_t sQ = base, sK = base + kTileBytes;
    float *sNegM = reinterpret_cast<float *>(gen + kTileBytes * (1 + kKStages)); // -(merged row max)
    float *sIl = sNegM + kMaxProbe;                                               // 1 / row sum
    int *sPos = reinterpret_cast<int *>(sIl + kMaxProbe);
    ScBarriers *bar = reinterpret_cast<ScBarriers *>(sPos + kMaxProbe);
    volatile int *abort_flag = &bar->abort_flag;

    // blockIdx.z = sequence of a batch: its own probe rows, statistics, column totals, counters
    // and scores, stacked; K of all sequences is one tensor map of n_seq * L rows
    const int chunk = blockIdx.x, h = blockIdx.y, g = h / a.G, z = blockIdx.z;
    q += z * a.q_seq;
    probe_pos += (long long)z * P;
    stats += (long long)z * a.Hq * n_chunks * kMaxProbe;
    accfx += (long long)z * a.L;
    counters += z * n_chunks;
    acc += (long long)z * a.L;
    norm += (long long)z * a.L;
    const int n_tiles_all = (a.L + kTile - 1) / kTile;
    const int t0 = chunk * tiles_per_chunk;
    const int t1 = min(n_tiles_all, t0 + tiles_per_chunk);
    const int n_tiles = t1 - t0;
    if (n_tiles <= 0) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar->q_full), 128);
        for (int s = 0; s < kKStages; ++s) {
            mbar_init(smem_u32(&bar->k_full[s]), 1);
            mbar_init(smem_u32(&bar->k_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar->s_full[b]), 1);
            mbar_init(smem_u32(&bar->s_empty[b]), 128);
        }
        bar->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 5) tmem_alloc(smem_u32(&bar->tmem_base), kTmemColsSc);
    // <0> may have been staged behind the caller's previous kernel: no global access before
    // that kernel is complete.  <1> only follows <0>, which triggers it at its very end, so
    // the inputs are settled; it waits further down, just before it reads <0>'s results.
    if (MODE == 0) grid_dependency_wait(q, probe_pos);
    else grid_launch_dependents();
    // probe positions
    if (threadIdx.x < kMaxProbe) {
        const int r = threadIdx.x;
        int c = (r < P) ? probe_pos[r] : -1;
        if (c >= a.L || (r < P && c < 0)) {
            if (chunk == 0 && h == 0 && MODE == 0) report(status_word, ZIPVL_DEV_BAD_INDEX);
            c = -1;
        }
        sPos[r] = c;
        // this thread's probe row is requested at once (it lands while the barriers and
        // the tensor memory are set up); the row is announced after the barrier below
        gather_row_sw128<(kHd >> 3)>(sQ, r, q + (long long)(c < 0 ? 0 : c) * a.q_stride + (long long)h * kHd, c >= 0);
        cp_async_commit();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bar->tmem_base;

    if (warp == 4) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            prefetch_tensormap(&kmap);
            for (int n = 0; n < n_tiles; ++n) {
                const int s = n % kKStages;
                if (n >= kKStages)
                    mbar_wait(smem_u32(&bar->k_empty[s]), ((n / kKStages) - 1) & 1, abort_flag);
                if (*abort_flag) break;
                const uint32_t fb = smem_u32(&bar->k_full[s]);
                // (head_dim 96: the second box runs 32 columns into the next head, or past the
                // row, where the copy fills zeros; no MMA reads those columns)
                mbar_expect_tx(fb, kHd > 64 ? kTileBytes : kHalfBytes);
                const uint32_t dst = sK + s * kTileBytes;
                const int y = z * a.L + (t0 + n) * kTile;
                tma_load_2d(dst, &kmap, g * kHd, y, fb);
                if (kHd > 64) tma_load_2d(dst + kHalfBytes, &kmap, g * kHd + 64, y, fb);
            }
        }
    } else if (warp == 5) {
        // ------------------------------ MMA issuer ---------------------------------
        // the whole warp runs the (warp-uniform) control flow so descriptors stay in
        // uniform registers; one elected lane issues
        const bool leader = elect_one();
        const uint32_t idesc = a.half ? idesc_f16kind(128, 128, false, false, false)
                                      : idesc_f16kind(128, 128, false, false, true);
        constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
        const uint32_t lo_q = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t lo_k0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
        mbar_wait(smem_u32(&bar->q_full), 0, abort_flag);
        for (int n = 0; n < n_tiles; ++n) {
            const int s = n % kKStages, b = n & 1;
            mbar_wait(smem_u32(&bar->k_full[s]), (n / kKStages) & 1, abort_flag);
            if (n >= 2) mbar_wait(smem_u32(&bar->s_empty[b]), ((n >> 1) - 1) & 1, abort_flag);
            tc_fence_after();
            const uint32_t lo_k = lo_k0 + s * (kTileBytes >> 4);
            if (leader) {
                if (!*abort_flag) {
#pragma unroll
                    for (int kb = 0; kb < kHd / 16; ++kb) {
                        const uint32_t o = ((kb >> 2) * kHalfBytes + (kb & 3) * 32) >> 4;
                        const uint64_t dq = ((uint64_t)kDescHi << 32) | (lo_q + o);
                        const uint64_t dk = ((uint64_t)kDescHi << 32) | (lo_k + o);
                        // stats: rows = probes; colsum: rows = keys
                        mma_ss(tmem + b * 128, MODE == 0 ? dq : dk, MODE == 0 ? dk : dq, idesc, kb > 0);
                    }
                }
                mma_commit(smem_u32(&bar->k_empty[s]));
                mma_commit(smem_u32(&bar->s_full[b]));
            }
            __syncwarp();
        }
    } else {
        // ------------------------------ consumers ----------------------------------
        const int row = threadIdx.x;  // TMEM lane: probe (stats) or key within tile (colsum)
        cp_async_wait<0>();          // the probe row requested before the set-up barrier
        fence_proxy_async();
        mbar_arrive(smem_u32(&bar->q_full));
        if (MODE == 1) {
            // Everything above (and the K loads and the first QK of the other warps) may
            // run while the statistics kernel is still finishing; its results are read
            // only behind this point.
            grid_dependency_wait(stats);
            const int r = row, c = sPos[row];
            float M = -INFINITY, Ls = 0.f;
            if (c >= 0) {
                // one pass over the chunk statistics, eight loads in flight (read through
                // L2: they were written while this kernel was already resident)
                const float2 *sp = stats + (long long)h * n_chunks * kMaxProbe + r;
                for (int c0 = 0; c0 < n_chunks; c0 += 8) {
                    float2 sv[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        sv[u] = (c0 + u < n_chunks) ? __ldcg(sp + (long long)(c0 + u) * kMaxProbe)
                                                    : make_float2(-INFINITY, 0.f);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (sv[u].y > 0.f) {
                            const float Mn = fmaxf(M, sv[u].x);
                            Ls = Ls * ex2(M - Mn) + sv[u].y * ex2(sv[u].x - Mn);
                            M = Mn;
                        }
                    }
                }
            }
            sNegM[r] = Ls > 0.f ? -M : 0.f;
            sIl[r] = Ls > 0.f ? 1.f / Ls : 0.f;
            consumer_barrier();         // the merged statistics of all 128 probes are in place
        }
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        const int my_pos = sPos[row];
        float m = -INFINITY, l = 0.f;
        for (int n = 0; n < n_tiles; ++n) {
            const int b = n & 1;
            const int j0 = (t0 + n) * kTile;
            mbar_wait(smem_u32(&bar->s_full[b]), (n >> 1) & 1, abort_flag);
            tc_fence_after();
            const uint32_t tS = lane_base + b * 128;
            // the whole 128-column row in registers: four loads, one wait; the TMEM
            // buffer is handed back to the MMA warp right away
            uint32_t sr[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, sr[c]);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(smem_u32(&bar->s_empty[b]));
            if (MODE == 0) {
                // visible keys of this probe row: j <= my_pos (and j < L)
                const int vis = min(my_pos, a.L - 1) - j0;  // last visible column, may be < 0
                if (vis >= 0) {
                    float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                    if (vis >= 127) {
#pragma unroll
                        for (int c = 0; c < 4; ++c)
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                mxa[e & 3] = fmaxf(mxa[e & 3], __uint_as_float(sr[c][e]));
                    } else {
#pragma unroll
                        for (int c = 0; c < 4; ++c)
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (c * 32 + e <= vis)
                                    mxa[e & 3] = fmaxf(mxa[e & 3], __uint_as_float(sr[c][e]));
                    }
                    const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3]));
                    const float m_new = fmaxf(m, mx * a.scale_log2);
                    l *= ex2(m - m_new);
                    m = m_new;
                    const float neg_m = -m;
                    float ps4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            const float p = ex2(fmaf(__uint_as_float(sr[c][e]), a.scale_log2, neg_m));
                            ps4[e & 3] += (c * 32 + e <= vis) ? p : 0.f;
                        }
                    l += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
                }
            } else {
                const int j = j0 + row;
                // first probe (ascending positions) that sees key j
                int first_vis;
                {
                    int lo = 0, hi = P;
                    while (lo < hi) {
                        const int mid = (lo + hi) >> 1;
                        if (sPos[mid] < j) lo = mid + 1; else hi = mid;
                    }
                    first_vis = lo;
                }
                // probes below the warp's first key see none of its keys: whole 32-probe chunks of
                // them are left out (probes ascend, the warp's rows too: lane 0 has the smallest bound)
                const int first_vis_warp = __shfl_sync(0xffffffffu, first_vis, 0);
                // ... and from the last lane's bound on every probe sees all of the warp's keys: no
                // test per element there.  Two elements per arithmetic instruction (packed fp32x2).
                const int all_vis_warp = __shfl_sync(0xffffffffu, first_vis, 31);
                const uint64_t scale2 = pack2f(a.scale_log2, a.scale_log2);
                const uint64_t *nm2 = reinterpret_cast<const uint64_t *>(sNegM);
                const uint64_t *il2 = reinterpret_cast<const uint64_t *>(sIl);
                uint64_t cs2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if ((c + 1) * 32 <= first_vis_warp) continue;
                    if (c * 32 >= all_vis_warp) {
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            const int pr = c * 32 + e;
                            float x0, x1;
                            unpack2f(fma2(pack2u(sr[c][e], sr[c][e + 1]), scale2, nm2[pr >> 1]), x0, x1);
                            cs2[(e >> 1) & 3] = fma2(pack2f(ex2(x0), ex2(x1)), il2[pr >> 1], cs2[(e >> 1) & 3]);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            const int pr = c * 32 + e;
                            // probes ascend, so "sees this key" is a prefix test on pr
                            float x0, x1;
                            unpack2f(fma2(pack2u(sr[c][e], sr[c][e + 1]), scale2, nm2[pr >> 1]), x0, x1);
                            const float p0 = (pr >= first_vis) ? ex2(x0) : 0.f;
                            const float p1 = (pr + 1 >= first_vis) ? ex2(x1) : 0.f;
                            cs2[(e >> 1) & 3] = fma2(pack2f(p0, p1), il2[pr >> 1], cs2[(e >> 1) & 3]);
                        }
                    }
                }
                float cs4[4];
                unpack2f(add2(cs2[0], cs2[1]), cs4[0], cs4[1]);
                unpack2f(add2(cs2[2], cs2[3]), cs4[2], cs4[3]);
                // the head's column sum goes into the column's fixed-point total (2^-40 units: a sum
                // of 128 probabilities per head stays far below 2^63): integer adds commute, so the
                // total does not depend on the order in which the heads arrive
                // (a sum that is not a number -- a NaN in a query or key row -- sets the total's top
                // bit, which no sum of the heads reaches: the column's scores come out as NaN)
                if (j < a.L) {
                    const float cs = (cs4[0] + cs4[1]) + (cs4[2] + cs4[3]);
                    if (cs == cs) atomicAdd(accfx + j, __float2ull_rn(cs * kFxScale));
                    else atomicOr(accfx + j, 1ull << 63);
                }
            }
        }
        if (MODE == 0)
            stats[((long long)h * n_chunks + chunk) * kMaxProbe + row] = make_float2(m, l);
    }

    // all work of this CTA is issued: the dependent kernel may be staged now, so its
    // launch latency overlaps the drain of this one
    if (MODE == 0) grid_launch_dependents();
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(status_word, ZIPVL_DEV_TIMEOUT);
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemColsSc);
    }
    if (MODE == 0) {
        // arm the per-chunk counter the column-sum kernel uses to find its last CTA, and clear
        // the chunk's column totals
        if (h == 0) {
            if (threadIdx.x == 0) counters[chunk] = 0;
            for (int j = t0 * kTile + (int)threadIdx.x; j < min(a.L, t1 * kTile); j += kThreadsSc) accfx[j] = 0ull;
        }
    } else {
        // The last head to finish a key chunk reads the totals of all heads (Eq. 6), normalises
        // (Eq. 8) and writes the scores: no extra launch, no float atomics.
        __shared__ int is_last;
        if (threadIdx.x == 0) {
            __threadfence();
            is_last = (atomicAdd(&counters[chunk], 1) == a.Hq - 1);
        }
        __syncthreads();
        if (is_last) {
            __threadfence();
            const int jlo = t0 * kTile, jhi = min(a.L, t1 * kTile);
            // probes with a position inside [0, L): ascending, so the valid ones are a
            // prefix of the shared-memory copy (invalid entries hold -1)
            int n_valid_probes = 0;
            {
                int lo = 0, hi = P;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (sPos[mid] >= 0) lo = mid + 1; else hi = mid;
                }
                n_valid_probes = lo;
            }
            for (int j = jlo + (int)threadIdx.x; j < jhi; j += kThreadsSc) {
                // the exact total of the heads' sums, rounded once
                const unsigned long long fx = __ldcg(accfx + j);
                const float sum = (fx >> 63) ? __int_as_float(0x7fc00000)
                                             : (float)((double)fx * (1.0 / (double)kFxScale));
                int lo = 0, hi = n_valid_probes;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (sPos[mid] < j) lo = mid + 1; else hi = mid;
                }
                const int nnz = n_valid_probes - lo;   // probes at positions j .. L-1
                acc[j] = sum;
                norm[j] = nnz > 0 ? sum / ((float)a.Hq * (float)nnz) : 0.f;
            }
        }
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

int tiles_per_chunk_for(int L, int Hq) {
    // all CTAs of a launch are resident at once: two per SM on 148 SMs, so at most
    // 296 / Hq key chunks per head
    const int n_tiles = (L + kTile - 1) / kTile;
    const int max_chunks = (Hq >= 296) ? 1 : 296 / Hq;
    int tpc = (n_tiles + max_chunks - 1) / max_chunks;
    if (tpc < 1) tpc = 1;
    return tpc;
}

}  // namespace

__global__ void sum_to_double_kernel(int L, const float *__restrict__ x, double *__restrict__ out);

bool score_tc_supported(const LayerArgs &a, int dtype, int n_probe) {
    return (dtype == ZIPVL_BF16 || dtype == ZIPVL_F16) && (a.D == 128 || a.D == 96 || a.D == 64) &&
           n_probe <= kMaxProbe &&
           encode_tiled_fn() != nullptr;
}

size_t score_tc_ws_bytes(int L, int Hq, int, int, int n_seq) {
    const int n_tiles = (L + kTile - 1) / kTile;
    const int tpc = tiles_per_chunk_for(L, Hq * n_seq);
    const size_t n_chunks = (n_tiles + tpc - 1) / tpc;
    size_t stats = (size_t)Hq * n_chunks * kMaxProbe * sizeof(float2);
    stats = (stats + 255) & ~(size_t)255;
    stats = ((stats * n_seq) + 255) & ~(size_t)255;
    const size_t totals = ((size_t)n_seq * L * sizeof(unsigned long long) + 255) & ~(size_t)255;
    return stats + totals + n_seq * n_chunks * sizeof(int);
}

zipvl_status launch_score_tc(const LayerArgs &a, const void *q, const void *k,
                             const int32_t *probe_pos, int P, float *acc, float *norm,
                             double *total, void *ws, int32_t *status_word, cudaStream_t st) {
    const int n_tiles = (a.L + kTile - 1) / kTile;
    const int tpc = tiles_per_chunk_for(a.L, a.Hq * a.n_seq);
    const int n_chunks = (n_tiles + tpc - 1) / tpc;
    size_t stats_bytes = (size_t)a.n_seq * a.Hq * n_chunks * kMaxProbe * sizeof(float2);
    stats_bytes = (stats_bytes + 255) & ~(size_t)255;
    float2 *stats = reinterpret_cast<float2 *>(ws);
    unsigned long long *accfx = reinterpret_cast<unsigned long long *>(reinterpret_cast<char *>(ws) + stats_bytes);
    const size_t totals_bytes = ((size_t)a.n_seq * a.L * sizeof(unsigned long long) + 255) & ~(size_t)255;
    int *counters = reinterpret_cast<int *>(reinterpret_cast<char *>(ws) + stats_bytes + totals_bytes);

    // tensor map over K viewed as [L rows, Hkv*d columns], box = 64 columns x 128 rows
    CUtensorMap kmap;
    // (a batch is stacked without gaps -- the caller checks -- so its K is one 2-D tensor)
    const cuuint64_t dims[2] = {(cuuint64_t)a.Hkv * a.D, (cuuint64_t)a.L * a.n_seq};
    const cuuint64_t strides[1] = {(cuuint64_t)a.kv_stride * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult cr = encode_tiled_fn()(&kmap, a.half ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                                          const_cast<void *>(k), dims, strides, box, estr,
                                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(ZIPVL_ERR_CUDA, "score: cuTensorMapEncodeTiled failed (%d)", (int)cr);

    const __nv_bfloat16 *qb = (const __nv_bfloat16 *)q;
    dim3 grid(n_chunks, a.Hq, a.n_seq);
    cudaError_t e = cudaSuccess;
    // both launches are programmatic dependents: <1> may begin its set-up, loads and first
    // MMA while <0> drains, and <0> itself may be staged behind the caller's previous kernel
#define ZIPVL_SCORE_LAUNCH(HD_)                                                                      \
    {                                                                                                \
        e = cudaFuncSetAttribute(score_tc_kernel<0, HD_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScSmem); \
        if (e == cudaSuccess)                                                                        \
            e = cudaFuncSetAttribute(score_tc_kernel<1, HD_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScSmem); \
        if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "score: smem opt-in: %s", cudaGetErrorString(e)); \
        e = launch_dependent(score_tc_kernel<0, HD_>, grid, dim3(kThreadsSc), kScSmem, st, kmap, a, qb, probe_pos, P, \
                             tpc, n_chunks, stats, accfx, counters, acc, norm, status_word);       \
        if (e == cudaSuccess)                                                                        \
            e = launch_dependent(score_tc_kernel<1, HD_>, grid, dim3(kThreadsSc), kScSmem, st, kmap, a, qb, probe_pos, \
                                 P, tpc, n_chunks, stats, accfx, counters, acc, norm, status_word); \
    }
    if (a.D == 128) ZIPVL_SCORE_LAUNCH(128)
    else if (a.D == 96) ZIPVL_SCORE_LAUNCH(96)
    else ZIPVL_SCORE_LAUNCH(64)
#undef ZIPVL_SCORE_LAUNCH
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "score: launch: %s", cudaGetErrorString(e));
    if (total)
        for (int z = 0; z < a.n_seq; ++z) sum_to_double_kernel<<<1, 1024, 0, st>>>(a.L, acc + (size_t)z * a.L, total + z);
    count_launches(total ? 2 + a.n_seq : 2);
    return check_launch("zipvl_score");
}

}  // namespace zipvl
