// Sparse causal prefill attention on the 5th-generation tensor cores
// (Algorithm 1: attention over Q[T], K[T], V[T]; Eq. 2 on the gathered tokens).
// 16-bit storage (bfloat16 or IEEE half), head_dim 128, fp32 softmax and
// accumulation, output in the storage type.
//
// One CTA = 256 gathered query rows of one head (two 128-row tiles A and B that
// share every key/value tile, which halves the shared-memory fill per flop);
// key/value tiles of 128 gathered tokens up to the diagonal.  Warp-specialised:
//   warps 0-3 / 4-7   softmax for tile A / tile B: thread = query row = TMEM
//              lane.  The exact row maximum of the tile is taken first, then
//              P = exp2(S*scale - m).  The running max m moves (and O is rescaled,
//              by warp vote) only when a tile's max outgrew it by more than 2^32
//              (2^8 for IEEE half); the storage type carries that range, so after
//              the first tile this is rare.  P goes back to tensor memory in the
//              storage type over S; at the end the thread normalises its row of O
//              and the warp stores whole 256-byte rows.
//   warps 8-11 producers: the index list drives the loads.  Sixteen lanes copy
//              one gathered 256-byte row with 16-byte async copies straight into
//              the 128-byte-swizzled layout the tensor core reads; K and V tiles
//              go through one ring of five 32 KB slots (K0 V0 K1 V1 ...).
//   warp 12    issues tcgen05.mma: S_X = Q_X K^T (shared-memory operands) and
//              O_X += P_X V (P from tensor memory, V as MN-major operand), the two
//              query tiles interleaved so the tensor pipe works on one while the
//              other is in softmax.  It looks at its barriers in turn and serves
//              whichever tile is ready.
//   warps 13-15 zero the rows of dropped tokens (PADDED output) while the attention
//              runs and, in the fused call, copy the CTA's own 256 K and V rows from
//              the last two ring tiles to the compacted cache.
// Tensor memory (512 columns): S_A | S_B | O_A | O_B, 128 fp32 columns each; P
// aliases the first 64 columns of its S.  Every wait is bounded; a wait that
// runs out sets ZIPVL_DEV_TIMEOUT and all roles unwind to the common exit.
#include <stdlib.h>
#include <string.h>

#include <type_traits>

#include "tc.cuh"
#include "tc_ptx.cuh"

namespace zipvl {
namespace {

using namespace ptx;

// (the shared-memory tiles are 128 columns wide; head_dim 64 and 96 use the front of them)
constexpr int kBM = 128, kBN = 128;   // query / key tile
constexpr int kPair = 2 * kBM;        // query rows per CTA
constexpr int kSlots = 5;             // ring of K / V tiles
constexpr int kWindow = 3;            // tile loads in flight per producer thread
constexpr int kHalfBytes = 128 * 128;        // 128 rows x 64 bf16 (one swizzle atom wide)
constexpr int kTileBytes = 2 * kHalfBytes;   // 128 rows x 128 bf16
constexpr int kThreadsTc = 512;       // four warpgroups: softmax A, softmax B, producers, MMA
constexpr int kRegsSoftmax = 200, kRegsOther = 56;
constexpr uint32_t kTmemCols = 512;
// the running max may lag a tile's max by this many octaves before O is rescaled: P stays
// below 2^32 (bfloat16 and fp32 carry that) or 2^8 (IEEE half tops out at 65504)
constexpr float kRescaleThreshold = 32.0f, kRescaleThresholdHalf = 8.0f;
// kept rows x query heads up to which the single-tile kernel is launched instead of this one
// (0: never by default -- it measured slower at every size tried, see the dispatch below)
constexpr long long kSingleTileMaxRows = 0;

struct Barriers {
    uint64_t q_full;
    uint64_t full[kSlots];
    uint64_t empty[kSlots];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t pv_done[2];
    uint64_t tail_full[2];   // the CTA's own key tiles (K and V) have landed: told by the issuer
    uint32_t tmem_base;
    int abort_flag;
};

constexpr size_t kSmemBytes = kTileBytes * (2 + kSlots) + sizeof(Barriers) + 1024;

// Gather 32 rows of 256 bytes into a swizzled tile with one warp.  Lane l holds
// the token of row (row0 + l) in my_tok (-1 = zero-fill); row0 is a multiple of 32
// and the tile is 1024-byte aligned.  Sixteen adjacent lanes copy one row (16 chunks
// of 16 B): lanes 0-15 row i, lanes 16-31 row i + 16, so every request covers whole
// 32-byte sectors of two rows.  The loop is the producers' whole instruction stream
// and they share their schedulers with the softmax warps, so it is kept to a
// shuffle, one multiply-add for the source, one xor for the swizzle and the copy.
template <bool kAllValid, int n_chunks16>
__device__ __forceinline__ void gather_rows32_impl(uint32_t tile, int row0, int my_tok,
                                                   const __nv_bfloat16 *base, unsigned int stride_bytes,
                                                   int lane) {
    const int c = lane & 15, sub = lane >> 4;
    // a row of head_dim 64 or 96 has 8 or 12 chunks: the other lanes copy nothing (zero-fill of
    // columns no MMA reads) and never look past the row
    const uint32_t lane_bytes = (n_chunks16 == 16 || c < n_chunks16) ? 16u : 0u;
    const char *src_lane = reinterpret_cast<const char *>(base) + ((n_chunks16 == 16 || c < n_chunks16) ? c : 0) * 16;
    // every term but the chunk is a multiple of 128: the swizzle is an xor of the low bits
    const uint32_t dst_lane = (tile + (row0 + 16 * sub) * 128 + (c >> 3) * kHalfBytes) | ((c & 7) << 4);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int t = __shfl_sync(0xffffffffu, my_tok, i, 16);        // row i of my half-warp
        const uint32_t dst = (dst_lane ^ ((i & 7) << 4)) + i * 128;
        if (kAllValid)
            cp_async16(dst, src_lane + (unsigned long long)(unsigned int)t * stride_bytes, lane_bytes);
        else
            cp_async16(dst, src_lane + (unsigned long long)(unsigned int)(t < 0 ? 0 : t) * stride_bytes,
                       t >= 0 ? lane_bytes : 0u);
    }
}
template <int n_chunks16>
__device__ __forceinline__ void gather_rows32(uint32_t tile, int row0, int my_tok,
                                              const __nv_bfloat16 *base, long long stride,
                                              int lane) {
    const unsigned int stride_bytes = (unsigned int)(stride * 2);     // (checked by the host: < 2^31)
    if (__all_sync(0xffffffffu, my_tok >= 0))
        gather_rows32_impl<true, n_chunks16>(tile, row0, my_tok, base, stride_bytes, lane);
    else
        gather_rows32_impl<false, n_chunks16>(tile, row0, my_tok, base, stride_bytes, lane);
}

// kHalf: the 16-bit storage type is IEEE half instead of bfloat16 (pointers are typed
// __nv_bfloat16 either way: only their width matters to the loads and stores)
// kHd: head_dim (64, 96 or 128), a compile-time constant so that the 128 instantiation carries
// none of the narrower rows' tests
template <bool kHalf, int kHd>
__global__ void __launch_bounds__(kThreadsTc, 1)
prefill_tc_kernel(LayerArgs a, const __nv_bfloat16 *__restrict__ q,
                  const __nv_bfloat16 *__restrict__ k, const __nv_bfloat16 *__restrict__ v,
                  const int32_t *__restrict__ idx, const int32_t *__restrict__ k_dev, int k_max,
                  __nv_bfloat16 *__restrict__ out, int out_mode, __nv_bfloat16 *__restrict__ kc,
                  __nv_bfloat16 *__restrict__ vc, int capacity, int32_t *__restrict__ len_out,
                  int32_t *status_word) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char *gen = smem_raw + (base - raw);
    const uint32_t sQ = base;                         // Q_A | Q_B
    const uint32_t sRing = base + 2 * kTileBytes;     // kSlots tiles
    Barriers *bar = reinterpret_cast<Barriers *>(gen + kTileBytes * (2 + kSlots));
    volatile int *abort_flag = &bar->abort_flag;

    // Set-up that needs no global memory comes first, so it overlaps the previous kernel's
    // drain when this one was staged early: barriers and the tensor-memory allocation.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_launch_dependents();
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar->q_full), 256);
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&bar->full[s]), 128);
            mbar_init(smem_u32(&bar->empty[s]), 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(smem_u32(&bar->s_full[x]), 1);
            mbar_init(smem_u32(&bar->p_full[x]), 128);
            mbar_init(smem_u32(&bar->pv_done[x]), 1);
            mbar_init(smem_u32(&bar->tail_full[x]), 1);
        }
        bar->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 12) tmem_alloc(smem_u32(&bar->tmem_base), kTmemCols);
    grid_dependency_wait(q, k, v, idx, k_dev);   // k_dev and idx are the previous kernel's output
    // grid.x = query head + Hq * sequence: every sequence of a batch has its own tensors, index
    // list, k, output and cache, stacked; its heaviest pairs still start first
    const int h = blockIdx.x % a.Hq, g = h / a.G;
    constexpr int nch = kHd >> 3;            // 16-byte chunks of a row
    {
        const int z = blockIdx.x / a.Hq;
        q += z * a.q_seq; k += z * a.kv_seq; v += z * a.kv_seq;
        idx += (long long)z * a.L;
        k_dev += z;
        out += (long long)z * (out_mode == ZIPVL_OUT_PADDED ? a.L : k_max) * a.Hq * kHd;
        if (kc != nullptr) {
            kc += (long long)z * capacity * a.Hkv * kHd;
            vc += (long long)z * capacity * a.Hkv * kHd;
            len_out += z;
        }
    }
    int n_valid = *k_dev;
    if (n_valid > k_max || n_valid < 0) {
        if (h == 0 && blockIdx.y == 0 && threadIdx.x == 0)
            report(status_word, ZIPVL_DEV_CAPACITY);
        n_valid = n_valid < 0 ? 0 : k_max;
    }
    // blocks are dispatched x-fastest: x = head, y = pair, so every head of the
    // heaviest (longest-diagonal) pair starts first -- longest-processing-time order.
    // The grid is sized by the host's bound k_max; the pairs past the actual k map to
    // the last rows of the grid and return at once.
    // An odd number of 128-row tiles leaves one tile without a partner.  That single is the
    // FIRST tile (one key tile: the cheapest item there is), and the pairs are (1,2), (3,4) ...;
    // were the pairs counted from the front, the single would be the last tile, a CTA that
    // walks the whole diagonal with one query tile and nothing to overlap its chain with.
    const int n_tiles = (n_valid + kBM - 1) / kBM;
    const int odd = n_tiles & 1;
    const int n_pairs = (n_tiles + 1) / 2;
    const int pt = n_pairs - 1 - (int)blockIdx.y;
    const int ta = pt > 0 ? 2 * pt - odd : 0;       // tile A of this CTA (tile B = ta + 1)
    const int q0 = ta * kBM;
    const bool no_work = (pt < 0 || q0 >= n_valid || (int)blockIdx.x >= a.Hq * a.n_seq);   // or a bad grid
    const bool has_b = !(odd && pt == 0) && (q0 + kBM) < n_valid;   // tile B exists and has a valid row
    const int n_a = ta + 1;                         // key tiles of A (diagonal = ta)
    const int n_kv = has_b ? n_a + 1 : n_a;         // key tiles of B (diagonal = ta + 1)

    // The first token index every loading thread needs is fetched before the set-up
    // barrier, so its latency hides behind it: a softmax thread's own query row, a
    // producer lane's row of key tile 0.
    auto token_of = [&](int i) {
        if (i >= n_valid) return -1;
        int t = idx[i];
        if (t < 0 || t >= a.L) { report(status_word, ZIPVL_DEV_BAD_INDEX); t = -1; }
        return t;
    };
    int first_tok = -1;
    if (!no_work) {
        if (warp < 8) first_tok = token_of(q0 + warp * 32 + lane);
        else if (warp < 12) first_tok = token_of((warp - 8) * 32 + lane);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bar->tmem_base;
    if (no_work) {                                  // a CTA past the kept set: give the columns back
        if (warp == 12) tmem_dealloc(tmem, kTmemCols);
        if (n_valid == 0 && blockIdx.y == 0 && (int)blockIdx.x < a.Hq * a.n_seq) {
            // nothing kept: the results are those of the two separate calls -- an all-zero
            // PADDED output (every row is a dropped token's) and a cache of length 0
            if (out_mode == ZIPVL_OUT_PADDED) {
                const uint4 z = make_uint4(0, 0, 0, 0);
                for (int e = threadIdx.x; e < a.L * 16; e += kThreadsTc)
                    if ((e & 15) < nch)
                        reinterpret_cast<uint4 *>(out + ((long long)(e >> 4) * a.Hq + h) * kHd)[e & 15] = z;
            }
            if (kc != nullptr && h == 0 && threadIdx.x == 0) *len_out = 0;
        }
        return;
    }

    if (warp >= 8 && warp < 12) {
        // ------------------------------ producers ------------------------------
        reg_dec<kRegsOther>();
        const int row0 = (warp - 8) * 32;   // this warp's 32 rows of every 128-row tile
        const int total = 2 * n_kv;         // K0 V0 K1 V1 ...
        int tok = first_tok;
        auto issue = [&](int seq) {
            const int slot = seq % kSlots;
            if ((seq & 1) == 0 && seq > 0) tok = token_of((seq >> 1) * kBN + row0 + lane);
            const __nv_bfloat16 *src = ((seq & 1) ? v : k) + (long long)g * kHd;
            gather_rows32<nch>(sRing + slot * kTileBytes, row0, tok, src, a.kv_stride, lane);
            cp_async_commit();
        };
        auto slot_free = [&](int seq, bool block) {
            if (seq < kSlots) return true;
            const uint32_t eb = smem_u32(&bar->empty[seq % kSlots]);
            const uint32_t par = ((seq / kSlots) - 1) & 1;
            if (block) { mbar_wait(eb, par, abort_flag); return true; }
            return warp_try_wait(eb, par);
        };
        // Loads are issued only into slots that are already free, so a landed tile is
        // never announced late because the thread sits waiting for a slot; the thread
        // blocks on a slot only when it has nothing in flight.
        // (The query rows are gathered by the softmax warps at the same time.)
        int issued = 0;
        for (int seq = 0; seq < total; ++seq) {
            while (issued < total && issued - seq < kWindow && slot_free(issued, issued == seq))
                issue(issued++);
            const int newer = issued - 1 - seq;     // groups younger than `seq` in flight
            if (newer >= 2) cp_async_wait<2>();
            else if (newer == 1) cp_async_wait<1>();
            else cp_async_wait<0>();
            fence_proxy_async();
            mbar_arrive(smem_u32(&bar->full[seq % kSlots]));
        }
    } else if (warp >= 12) {
        // ---------------------- MMA issuer (warp 12), zero-fill (13-15) ----------------------
        reg_dec<kRegsOther>();
        if (warp > 12) {
            // PADDED output: the rows of dropped tokens in front of each kept token of this
            // CTA's 256 rows (and behind the very last kept token) are zeroed by these three
            // otherwise idle warps while the attention runs, off the critical path.  A lane
            // looks up the gap in front of one kept token; the warp then clears the gaps one
            // after another, two 256-byte rows per step.
            if (out_mode == ZIPVL_OUT_PADDED) {
                const uint4 z = make_uint4(0, 0, 0, 0);
                const int sub = lane >> 4, ch = lane & 15;
                auto clear_rows = [&](int r0, int r1) {
                    if (ch < nch)
                        for (int zr = r0 + sub; zr < r1; zr += 2)
                            reinterpret_cast<uint4 *>(out + ((long long)zr * a.Hq + h) * kHd)[ch] = z;
                };
                for (int i0 = (warp - 13) * 32; i0 < (has_b ? kPair : kBM); i0 += 3 * 32) {
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
            // Fused KV compaction (Algorithm 1: K = K[T], V = V[T]).  The last key tiles a CTA
            // loads -- its tile A and, if it has one, its tile B -- hold exactly the K and V rows of its
            // own 256 kept tokens, already gathered into shared memory for the attention.  The
            // CTA of the first query head of a KV group writes them to the compacted cache
            // from there (every (pair, kv head) once over the grid): these warps wait for the
            // tile like the issuer does and un-swizzle it, two rows per instruction.  The
            // slots of a CTA's last tiles are never refilled, so there is no race with the
            // producers; the attention only reads them.
            if (kc != nullptr && h % a.G == 0) {
                const int lim = min(n_valid, capacity);
                const int sub = lane >> 4, ch = lane & 15;
                for (int j = ta; j < n_kv; ++j) {               // key tile j = kept tokens 128j ..
                    // the issuer follows the ring in order and says when K and V of this tile
                    // are in (the ring's own barriers are only meaningful to a reader that
                    // keeps up with every phase)
                    mbar_wait(smem_u32(&bar->tail_full[j - ta]), 0, abort_flag);
                    for (int kind = 0; kind < 2; ++kind) {       // 0: K (group 2j), 1: V (group 2j+1)
                        const int seq = 2 * j + kind;
                        const unsigned char *tile = gen + (size_t)kTileBytes * (2 + seq % kSlots);
                        __nv_bfloat16 *dstc = kind ? vc : kc;
                        for (int r = (warp - 13) * 2 + sub; r < kBN; r += 3 * 2) {
                            const int i = j * kBN + r;
                            if (i >= lim || ch >= nch) continue;    // (a row with an invalid index is all zeros here)
                            const uint4 w = *reinterpret_cast<const uint4 *>(
                                tile + (ch >> 3) * kHalfBytes + r * 128 + (((ch & 7) ^ (r & 7)) << 4));
                            reinterpret_cast<uint4 *>(dstc + ((long long)i * a.Hkv + g) * kHd)[ch] = w;
                        }
                    }
                }
                if (h == 0 && blockIdx.y == 0 && warp == 13 && lane == 0) {
                    *len_out = lim;
                    if (n_valid > capacity) report(status_word, ZIPVL_DEV_CAPACITY);
                }
            }
        }
        if (warp == 12) {
            // The whole warp runs the control flow (so every operand is warp-uniform
            // and stays in uniform registers); one elected lane issues.
            const bool leader = elect_one();
            constexpr uint32_t idesc_qk = idesc_f16kind(kBM, kBN, false, false, !kHalf);
            constexpr uint32_t idesc_pv = idesc_f16kind(kBM, kHd, false, true, !kHalf);   // N = head_dim
            // Descriptors are built once: the high word is constant (SBO 1024 B,
            // version, 128-byte swizzle); the low word is (address >> 4) | LBO << 16
            // and moves by a compile-time offset per k-block, so issuing one MMA is
            // one add and the instruction itself.
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t lo_q0 = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t lo_ring = (sRing & 0x3FFFFu) >> 4;
            auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
            auto wait_full = [&](int seq) {
                mbar_wait(smem_u32(&bar->full[seq % kSlots]), (seq / kSlots) & 1, abort_flag);
                tc_fence_after();
            };
            auto release = [&](int seq) { if (leader) mma_commit(smem_u32(&bar->empty[seq % kSlots])); };
            // S_x = Q_x K(n)^T
            auto qk = [&](int x, int n) {
                const uint32_t lo_k = (lo_ring + ((2 * n) % kSlots) * (kTileBytes >> 4)) | (1u << 16);
                const uint32_t lo_q = lo_q0 + x * (kTileBytes >> 4);
                const uint32_t d = tmem + x * 128;
                if (leader) {
#pragma unroll
                    for (int kb = 0; kb < kHd / 16; ++kb) {
                        const uint32_t o = ((kb >> 2) * kHalfBytes + (kb & 3) * 32) >> 4;
                        mma_ss(d, desc(lo_q + o), desc(lo_k + o), idesc_qk, kb > 0);
                    }
                    mma_commit(smem_u32(&bar->s_full[x]));
                }
                __syncwarp();
            };
            // O_x += P_x V(n): P from tensor memory, V MN-major (LBO = one 64-column half)
            auto pv = [&](int x, int n) {
                const uint32_t lo_v = (lo_ring + ((2 * n + 1) % kSlots) * (kTileBytes >> 4)) |
                                      ((uint32_t)(kHalfBytes >> 4) << 16);
                const uint32_t d = tmem + 256 + x * 128, p = tmem + x * 128;
                if (leader) {
#pragma unroll
                    for (int kb = 0; kb < kBN / 16; ++kb)
                        mma_ts(d, p + kb * 8, desc(lo_v + kb * (2048 >> 4)), idesc_pv, (n > 0 || kb > 0));
                }
                __syncwarp();
            };
            mbar_wait(smem_u32(&bar->q_full), 0, abort_flag);
            wait_full(0);
            if (!*abort_flag) {
                qk(0, 0);
                if (has_b) qk(1, 0);
            }
            release(0);
            // The two query tiles advance independently: whichever has its P ready
            // (and its V / next K tile landed) is served; nothing blocks on the other.
            // A ring slot is released by whichever tile uses it last.
            int next[2] = {0, 0};
            bool loads_ok[2] = {false, false};
            const int cnt[2] = {n_a, has_b ? n_kv : 0};
            auto is_full = [&](int seq) {
                return warp_try_wait(smem_u32(&bar->full[seq % kSlots]), (seq / kSlots) & 1);
            };
            for (uint32_t spin = 0; (next[0] < cnt[0] || next[1] < cnt[1]) && !*abort_flag; ++spin) {
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    const int n = next[x], o = 1 - x;
                    if (n >= cnt[x]) continue;
                    const bool more = (n + 1 < cnt[x]);
                    // the tiles this step reads are looked up while the issuer is idle, so
                    // a finished softmax finds the way to the tensor pipe already clear
                    if (!loads_ok[x]) {
                        // (every producer thread announces its tiles in order, so a landed
                        // K(n+1) says that V(n) has landed too: one look at one barrier)
                        loads_ok[x] = is_full(more ? 2 * n + 2 : 2 * n + 1);
                        if (!loads_ok[x]) continue;
                        // The last step of tile A reads the key tile of A's own tokens, that of
                        // tile B the one of B's -- the CTA's own 256 tokens: K and V of that tile are in now,
                        // which the warps that copy them to the compacted cache are told here
                        // (once per tile: loads_ok is set once per step).
                        if (!more && leader) mbar_arrive(smem_u32(&bar->tail_full[x]));
                    }
                    if (!warp_try_wait(smem_u32(&bar->p_full[x]), n & 1)) continue;
                    tc_fence_after();
                    pv(x, n);
                    // the commit behind QK(n+1) also covers PV(n): a landed S(n+1) tells the
                    // softmax warps that O is complete through tile n; the last PV commits itself
                    if (more) qk(x, n + 1);
                    else if (leader) mma_commit(smem_u32(&bar->pv_done[x]));
                    next[x] = n + 1;
                    loads_ok[x] = false;
                    // V(n): the other tile is past it, or never uses it
                    if (!(n < cnt[o]) || next[o] > n) release(2 * n + 1);
                    // K(n+1): released once every user has issued its QK
                    if (more && (!(n + 1 < cnt[o]) || next[o] > n)) release(2 * n + 2);
                    spin = 0;
                }
                if (spin >= kWaitLimit) *abort_flag = 1;
            }
        }
    } else {
        // --------------------------- softmax / epilogue ---------------------------
        reg_inc<kRegsSoftmax>();
        const int x = warp >> 2;                        // 0 = tile A, 1 = tile B
        const int row = threadIdx.x & 127;              // TMEM lane, query row in tile
        // every warp gathers its own 32 query rows (rows past the kept set are zero-filled)
        gather_rows32<nch>(sQ + x * kTileBytes, (warp & 3) * 32, first_tok, q + (long long)h * kHd, a.q_stride,
                           lane);
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        mbar_arrive(smem_u32(&bar->q_full));
        const int n_mine = (x == 0) ? n_a : n_kv;
        const int diag_tile = ta + x;
        if (x == 0 || has_b) {
            const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
            const uint32_t tS = lane_base + x * 128;
            const uint32_t tO = lane_base + 256 + x * 128;
            float m = -INFINITY, l = 0.f;
            const uint64_t scale2 = pack2f(a.scale_log2, a.scale_log2);
            // One key tile of one query row per thread.  The exact row maximum of the
            // tile comes first, so every exponential is taken against a settled max and
            // P can be stored chunk by chunk while the next chunk is computed.  The
            // running max m is only moved when the tile's max outgrew it by more than 2^32
            // (P then stays below 2^32, far inside bf16 and fp32 range), which makes the
            // read-modify-write of O a rare event.
            const int quad = warp & 3;                  // this warp's 32-row (and, on the diagonal, 32-column) block
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
                // 32-column chunk: chunks below it are fully visible, the chunk with the
                // warp's own index is cut per lane (column e <= lane), chunks above it are
                // fully masked -- three warp-uniform cases instead of a test per element.
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
                        // a fully masked chunk: P = 0, no exponentials
#pragma unroll
                        for (int e = 0; e < 16; ++e) p16[e] = 0u;
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
                    // P (bf16) overwrites the front of S: every S column is in registers
                    tmem_st16(tS + c * 16, p16);
                }
                float sa, sb, sc, sd;
                unpack2f(add2(sum2[0], sum2[1]), sa, sb);
                unpack2f(add2(sum2[2], sum2[3]), sc, sd);
                l = l * alpha + ((sa + sb) + (sc + sd));
                if (rescale) {
                    // O is complete through tile n-1: the commit that announced S(n) was
                    // issued after PV(n-1) and covers it
#pragma unroll 1
                    for (int c = 0; c < (kHd >> 5); ++c) {
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
            for (int n = 0; n < n_mine; ++n) {
                mbar_wait(smem_u32(&bar->s_full[x]), n & 1, abort_flag);
                tc_fence_after();
                if (n == diag_tile) tile(std::true_type{}, n);
                else tile(std::false_type{}, n);
                tc_fence_before();
                mbar_arrive(smem_u32(&bar->p_full[x]));
            }
            // ---- epilogue: O / l -> bf16 -> global ----
            mbar_wait(smem_u32(&bar->pv_done[x]), 0, abort_flag);   // committed once, behind the last PV
            tc_fence_after();
            const int i = q0 + x * kBM + row;
            const int t = first_tok;
            const float inv = l > 0.f ? 1.f / l : 0.f;
            const bool padded = (out_mode == ZIPVL_OUT_PADDED);
            __nv_bfloat16 *dst = nullptr;
            if (t >= 0 && !*abort_flag)
                dst = out + ((long long)(padded ? t : i) * a.Hq + h) * kHd;
            // The normalised row goes to global memory through this tile's query buffer
            // (no MMA reads it any more: the last score tile has landed).  Each warp stages
            // its own 32 rows -- a lane writes its row, 16-byte chunks XOR-swizzled by the row
            // so that neither side has bank conflicts -- and then writes them out two rows
            // per instruction, 16 lanes covering one contiguous 256-byte row.
            unsigned char *stage = gen + (size_t)x * kTileBytes + (size_t)(warp & 3) * (32 * 256);
#pragma unroll 1
            for (int c = 0; c < (kHd >> 5); ++c) {
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
                    // destination of row rr of this warp: its lane holds the pointer
                    const unsigned long long d = __shfl_sync(0xffffffffu, (unsigned long long)dst, rr);
                    const uint4 w = *reinterpret_cast<const uint4 *>(stage + rr * 256 + ((ch ^ (rr & 15)) << 4));
                    if (d && ch < nch) reinterpret_cast<uint4 *>(d)[ch] = w;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(status_word, ZIPVL_DEV_TIMEOUT);
    if (warp == 12) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace

bool prefill_tc_supported(const LayerArgs &a, int dtype) {
    // (row strides in bytes are kept in 32 bits by the gathers)
    return (dtype == ZIPVL_BF16 || dtype == ZIPVL_F16) && (a.D == 128 || a.D == 96 || a.D == 64) &&
           a.q_stride < (1ll << 30) &&
           a.kv_stride < (1ll << 30);
}

size_t prefill_tc_ws_bytes(int, int, int, int) { return 0; }

zipvl_status launch_prefill_tc(const LayerArgs &a, const void *q, const void *k, const void *v,
                               const int32_t *idx, const int32_t *k_dev, int k_max, void *out,
                               int out_mode, void *k_cache, void *v_cache, int capacity,
                               int32_t *len_out, void *ws, int32_t *status_word, cudaStream_t st) {
    (void)ws;
    // The kernel with one 128-row query tile per CTA and two CTAs per SM (prefill_tc1.cu) has
    // smaller work items and hides a CTA's prologue and epilogue behind its neighbour, but
    // every key / value tile then feeds one query tile instead of two, and with room for
    // only one K and one V buffer its loads (2500-3400 cycles per tile next to busy softmax
    // warps) sit on the critical path of each step: 94 against 72 microseconds on the
    // 2944-token, 32-head layer, 829 against 1147 TFLOP/s on the 18432-token one.  It gives
    // the same bits and stays selectable with ZIPVL_PREFILL_KERNEL=single (pair = this one).
    const char *env = getenv("ZIPVL_PREFILL_KERNEL");
    const int forced = !env ? 0 : (!strcmp(env, "pair") ? 1 : (!strcmp(env, "single") ? 2 : 0));
    const bool single = forced ? (forced == 2) : ((long long)k_max * a.Hq <= kSingleTileMaxRows);
    if (single && a.n_seq == 1 && a.D == 128)
        return launch_prefill_tc1(a, q, k, v, idx, k_dev, k_max, out, out_mode, k_cache, v_cache,
                                  capacity, len_out, status_word, st);
    auto kernel = a.half ? prefill_tc_kernel<true, 128> : prefill_tc_kernel<false, 128>;
    if (a.D == 96) kernel = a.half ? prefill_tc_kernel<true, 96> : prefill_tc_kernel<false, 96>;
    if (a.D == 64) kernel = a.half ? prefill_tc_kernel<true, 64> : prefill_tc_kernel<false, 64>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess)
        return fail(ZIPVL_ERR_CUDA, "sparse_prefill: smem opt-in: %s", cudaGetErrorString(e));
    dim3 grid(a.Hq * a.n_seq, (k_max + kPair - 1) / kPair);
    e = launch_dependent(kernel, grid, dim3(kThreadsTc), kSmemBytes, st, a, (const __nv_bfloat16 *)q,
                         (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, idx, k_dev, k_max,
                         (__nv_bfloat16 *)out, out_mode, (__nv_bfloat16 *)k_cache,
                         (__nv_bfloat16 *)v_cache, capacity, len_out, status_word);
    if (e != cudaSuccess)
        return fail(ZIPVL_ERR_CUDA, "sparse_prefill: launch: %s", cudaGetErrorString(e));
    count_launches(1);
    return check_launch("zipvl_sparse_prefill");
}

}  // namespace zipvl
