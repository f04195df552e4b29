// Grouped-query decode over the kept cache on the 5th-generation tensor cores
// (Algorithm 2; Eq. 4 append, Eq. 5 attention of one query token over the whole cache).
// 16-bit storage, head_dim 64, 96 or 128, 2 to 32 query heads per key/value head.
//
// With G query heads sharing one cached row, the CUDA-core kernel needs 2*G multiply-adds per
// cached element; from G = 4 on that, not HBM, sets its pace.  Here the G query rows of a
// kv head are the rows of an MMA tile, so every cached byte is still read once and the
// arithmetic moves to the tensor pipe.
//
// CTA = (chunk of cache rows, kv head, request); key/value tiles of 128 rows.
//   warps 0-3  softmax.  The tile has 128 rows and only G are needed, so the G query rows are
//              loaded FOUR times: at rows 32w .. 32w+G-1 for w = 0..3.  Copy w (the lanes of warp
//              w, which owns TMEM lanes 32w..32w+31) takes the keys 32w..32w+31 of every tile
//              and leaves P = 0 for the others, so the four warps (one per scheduler and exp2
//              unit) share a tile's columns and each keeps its own running (max, sum) and its
//              own rows of O; the four are merged at the end.  Rows no copy uses hold whatever
//              shared memory held: a row of an MMA result depends on its own row of A only.
//   warps 4..  producers (groups of four warps): 16 lanes copy one cached row (256 B) with 16-byte async copies into
//              the 128-byte-swizzled tile; K and V tiles go through one ring of six 32 KB slots.
//              Rows behind the request's length are zero-filled and flagged (one bit per row).
//              The appended row (Eq. 4) is taken from k_new / v_new and stored into the cache.
//   last warp  issues tcgen05.mma: S = Q K^T (shared-memory operands) into one of two S buffers,
//              O += P V (P from tensor memory, V as MN-major operand).
// Tensor memory (512 columns): S0 | S1 | P0 P1 (64 each) | O.
// Each CTA leaves one (m, l, o[128]) per query head in the workspace, in the layout the merge
// kernel of the CUDA-core path reads.  Every wait is bounded.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace zipvl {
namespace {

using namespace ptx;

constexpr int kD = 128, kBN = 128;
constexpr int kSlots = 6;              // ring of K / V tiles (K0 V0 K1 V1 K2 V2)
// Producer warps come in groups of four (one group fills one tile: a warp per 32 rows).  A warp
// can only have so many 16-byte async copies outstanding, so the bytes in flight -- and with
// them the bandwidth the SM can draw -- grow with the number of producer warps, not with the
// depth of one warp's queue: four warps alone stay near 11 bytes per clock.  Group j takes the
// tiles j, j + kGroups, ... of the ring sequence K0 V0 K1 V1 ...
#ifndef ZIPVL_DT_GROUPS
#define ZIPVL_DT_GROUPS 3
#endif
constexpr int kGroups = ZIPVL_DT_GROUPS;
// (every use of a ring slot must fall to the same group, which fills its tiles in order: a
// slot's "empty" barrier is then never more than one phase behind its reader)
static_assert(6 % ZIPVL_DT_GROUPS == 0, "a group owns whole ring slots");
#ifndef ZIPVL_DT_WINDOW
#define ZIPVL_DT_WINDOW 3
#endif
constexpr int kWindow = ZIPVL_DT_WINDOW;             // tile loads in flight per producer thread
constexpr int kIssuerWarp = 4 + 4 * kGroups;
constexpr int kHalfBytes = 128 * 128;
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kThreadsDt = 32 * (kIssuerWarp + 1);   // 4 softmax warps, the producer warps, 1 issuer warp
constexpr uint32_t kTmemColsDt = 512;
constexpr uint32_t kColS = 0, kColP = 256, kColO = 384;
constexpr int kMaxGroup = 32;
#ifndef ZIPVL_DT_MAXTPC
#define ZIPVL_DT_MAXTPC 16
#endif
constexpr int kMaxTilesPerChunk = ZIPVL_DT_MAXTPC;
constexpr float kRescaleBf16 = 32.0f, kRescaleHalf = 8.0f;   // octaves the running max may lag

struct DtBarriers {
    uint64_t q_full;
    uint64_t full[kSlots];
    uint64_t empty[kSlots];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t pv_done;                  // once per tile, behind PV(n)
    uint64_t o_final;                  // once, behind the last PV
    uint32_t tmem_base;
    int abort_flag;
    uint32_t valid[8][4];              // per key tile (mod 8) and 32-row block: rows that count
};

// merged at the end: (m, l) and o[128] of the four column quarters of every query head
struct DtMerge {
    float m[4][kMaxGroup], l[4][kMaxGroup];
    float o[4][kMaxGroup][kD + 1];     // (+1: the lanes of a warp write different banks)
};

constexpr size_t kDtSmem = kTileBytes * (1 + kSlots) + sizeof(DtBarriers) + 1024;
static_assert(sizeof(DtMerge) <= kTileBytes * kSlots, "the merge staging reuses the ring");

// HD: head_dim (64, 96 or 128); the shared-memory tiles stay 128 wide and the narrower heads use
// the front of them
template <bool kHalf, bool kPaged, int HD>
__global__ void __launch_bounds__(kThreadsDt, 1)
decode_tc_kernel(int Hq, int Hkv, float scale_log2, const __nv_bfloat16 *__restrict__ q,
                 const __nv_bfloat16 *__restrict__ k_new, const __nv_bfloat16 *__restrict__ v_new,
                 __nv_bfloat16 *__restrict__ k_cache, __nv_bfloat16 *__restrict__ v_cache,
                 const int64_t *__restrict__ cache_off, PageArgs pg,
                 const int32_t *__restrict__ capacity, int32_t *__restrict__ seq_lens, int max_len,
                 int chunk, int n_chunks, float *__restrict__ ws, int *__restrict__ lens,
                 int32_t *status_word) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char *gen = smem_raw + (base - raw);
    const uint32_t sQ = base;
    const uint32_t sRing = base + kTileBytes;
    DtBarriers *bar = reinterpret_cast<DtBarriers *>(gen + kTileBytes * (1 + kSlots));
    volatile int *abort_flag = &bar->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    grid_launch_dependents();
    // lengths and caches may be the previous kernel's output
    grid_dependency_wait(q, k_new, v_new, k_cache, v_cache, cache_off, capacity, seq_lens, pg.table);
    const int G = Hq / Hkv;
    const int g = blockIdx.y, b = blockIdx.z;
    const int h0 = g * G;                    // first query head of this kv head
    const bool first = blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0;

    // Eq. 4: the new row goes to position seq_lens[b] if the cache has room.  A request whose
    // length is negative or beyond its capacity, or whose cache offset breaks the 16-byte
    // alignment of the row copies, is skipped as a whole and reported.
    const int old_len = seq_lens[b];
    const int cap = capacity[b];
    const long long coff = kPaged ? 0ll : cache_off[b];
    const bool bad = old_len < 0 || old_len > cap || ((coff * 2) & 15) != 0;
    if (bad && first) report(status_word, ZIPVL_DEV_BAD_INDEX);
    const bool appended = !bad && k_new != nullptr && old_len < cap;
    if (k_new != nullptr && !bad && !appended && first) report(status_word, ZIPVL_DEV_CAPACITY);
    int len = bad ? 0 : old_len + (appended ? 1 : 0);
    if (len > max_len) {
        if (first) report(status_word, ZIPVL_DEV_CAPACITY);
        len = max_len;
    }
    const int new_row = appended ? old_len : -1;
    // the length this step attends over, for the merge kernel (which must not read seq_lens: it
    // also writes it)
    if (first) {
        lens[2 * b] = len;
        lens[2 * b + 1] = appended ? 1 : 0;
    }
    const int c0 = blockIdx.x * chunk;
    if (c0 >= len) {
        // a chunk past the request's length: empty partials (the merge reads every chunk slot)
        if ((int)threadIdx.x < G) {
            float *dst = ws + (((long long)b * Hq + h0 + threadIdx.x) * n_chunks + blockIdx.x) * (HD + 2);
            dst[0] = -INFINITY;
            dst[1] = 0.f;
        }
        return;
    }
    const int c1 = min(len, c0 + chunk);
    const int n_tiles = (c1 - c0 + kBN - 1) / kBN;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar->q_full), 128);
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&bar->full[s]), 128);
            mbar_init(smem_u32(&bar->empty[s]), 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(smem_u32(&bar->s_full[x]), 1);
            mbar_init(smem_u32(&bar->p_full[x]), 128);
        }
        mbar_init(smem_u32(&bar->pv_done), 1);
        mbar_init(smem_u32(&bar->o_final), 1);
        bar->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == kIssuerWarp) tmem_alloc(smem_u32(&bar->tmem_base), kTmemColsDt);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bar->tmem_base;
    const long long row_pitch = (long long)Hkv * HD;          // elements between cache rows

    if (warp >= 4 && warp < kIssuerWarp) {
        // ------------------------------ producers ------------------------------
        const int p = (warp - 4) & 3;           // this warp's 32 rows of every 128-row tile
        const int group = (warp - 4) >> 2;
        const int c = lane & 15, sub = lane >> 4;
        const int32_t *my_table = kPaged ? pg.table + (long long)b * pg.stride : nullptr;
        const __nv_bfloat16 *new_k = k_new ? k_new + ((long long)b * Hkv + g) * HD : nullptr;
        const __nv_bfloat16 *new_v = v_new ? v_new + ((long long)b * Hkv + g) * HD : nullptr;
        const long long head_off = coff + (long long)g * HD;
        long long my_off = -1;                  // cache offset (elements) of row 32p + lane of the tile
        const int total = 2 * n_tiles;          // K0 V0 K1 V1 ...
        // this group's share of the sequence: seq = group + j * kGroups
        const int mine_n = group < total ? (total - group + kGroups - 1) / kGroups : 0;
        auto issue = [&](int seq) {
            const int n = seq >> 1, kind = seq & 1;
            const int j0 = c0 + n * kBN;
            {
                // one lane per row: where the row lives (-1: behind the length, or in a page
                // outside the pool, which is reported and left out of the attention)
                const int row = j0 + p * 32 + lane;
                my_off = -1;
                if (row < c1) {
                    if (!kPaged) {
                        my_off = row * row_pitch;
                    } else {
                        const int page = my_table[row >> pg.shift];
                        if (page < 0 || page >= pg.n_pages) { if (kind == 0) report(status_word, ZIPVL_DEV_BAD_INDEX); }
                        else my_off = (((long long)page << pg.shift) + (row & ((1 << pg.shift) - 1))) * row_pitch;
                    }
                }
                const uint32_t word = __ballot_sync(0xffffffffu, my_off >= 0);
                if (lane == 0 && kind == 0) bar->valid[n & 7][p] = word;
            }
            const uint32_t tile = sRing + (seq % kSlots) * kTileBytes;
            __nv_bfloat16 *cache = kind ? v_cache : k_cache;
            const __nv_bfloat16 *fresh = kind ? new_v : new_k;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int r = p * 32 + i + 16 * sub;                    // row of the tile
                const long long off = __shfl_sync(0xffffffffu, my_off, i + 16 * sub);
                const uint32_t dst = tile + r * 128 + (c >> 3) * kHalfBytes + (((c & 7) ^ (r & 7)) << 4);
                const bool ok = off >= 0;
                const bool piece = c < HD / 8;                          // (a row has HD / 8 chunks of 16 bytes)
                const __nv_bfloat16 *src = cache + (ok ? off : 0) + head_off + (piece ? c : 0) * 8;
                if (ok && j0 + r == new_row) {
                    // the appended token: read from k_new / v_new, stored into the cache on the way
                    src = fresh + (piece ? c : 0) * 8;
                    if (piece)
                        *reinterpret_cast<uint4 *>(cache + off + head_off + c * 8) =
                            *reinterpret_cast<const uint4 *>(src);
                }
                cp_async16(dst, src, (ok && piece) ? 16u : 0u);
            }
            cp_async_commit();
        };
        auto slot_free = [&](int seq, bool block) {
            if (seq < kSlots) return true;
            const uint32_t eb = smem_u32(&bar->empty[seq % kSlots]);
            const uint32_t par = ((seq / kSlots) - 1) & 1;
            if (block) { mbar_wait(eb, par, abort_flag); return true; }
            return warp_try_wait(eb, par);
        };
        // loads go only into slots that are already free; the thread blocks on a slot only
        // when it has nothing in flight
        int issued = 0;
        for (int j = 0; j < mine_n; ++j) {
            const int seq = group + j * kGroups;
            while (issued < mine_n && issued - j < kWindow && slot_free(group + issued * kGroups, issued == j)) {
                issue(group + issued * kGroups);
                ++issued;
            }
            const int newer = issued - 1 - j;       // groups younger than this one in flight
            if (newer >= 2) cp_async_wait<2>();
            else if (newer == 1) cp_async_wait<1>();
            else cp_async_wait<0>();
            fence_proxy_async();
            mbar_arrive(smem_u32(&bar->full[seq % kSlots]));
        }
    } else if (warp == kIssuerWarp) {
        // ------------------------------ MMA issuer ------------------------------
        const bool leader = elect_one();
        constexpr uint32_t idesc_qk = idesc_f16kind(128, kBN, false, false, !kHalf);
        constexpr uint32_t idesc_pv = idesc_f16kind(128, HD, false, true, !kHalf);
        constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
        const uint32_t lo_q = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t lo_ring = (sRing & 0x3FFFFu) >> 4;
        auto desc = [](uint32_t lo) { return ((uint64_t)kDescHi << 32) | lo; };
        auto wait_full = [&](int seq) {
            mbar_wait(smem_u32(&bar->full[seq % kSlots]), (seq / kSlots) & 1, abort_flag);
            tc_fence_after();
        };
        // S(n) = Q K(n)^T into buffer n & 1; the commits free K's slot and announce S
        auto qk = [&](int n) {
            const int seq = 2 * n;
            wait_full(seq);
            const uint32_t lo_k = (lo_ring + (seq % kSlots) * (kTileBytes >> 4)) | (1u << 16);
            const uint32_t d = tmem + kColS + (n & 1) * 128;
            if (leader && !*abort_flag) {
#pragma unroll
                for (int kb = 0; kb < HD / 16; ++kb) {
                    const uint32_t o = ((kb >> 2) * kHalfBytes + (kb & 3) * 32) >> 4;
                    mma_ss(d, desc(lo_q + o), desc(lo_k + o), idesc_qk, kb > 0);
                }
            }
            if (leader) {
                mma_commit(smem_u32(&bar->empty[seq % kSlots]));
                mma_commit(smem_u32(&bar->s_full[n & 1]));
            }
            __syncwarp();
        };
        mbar_wait(smem_u32(&bar->q_full), 0, abort_flag);
        tc_fence_after();
        qk(0);
        if (n_tiles > 1) qk(1);
        for (int n = 0; n < n_tiles; ++n) {
            // P(n) is written: softmax(n) is also done reading S(n), so QK(n+2) may reuse it
            mbar_wait(smem_u32(&bar->p_full[n & 1]), (n >> 1) & 1, abort_flag);
            const int seq = 2 * n + 1;
            wait_full(seq);
            const uint32_t lo_v = (lo_ring + (seq % kSlots) * (kTileBytes >> 4)) |
                                  ((uint32_t)(kHalfBytes >> 4) << 16);
            const uint32_t d = tmem + kColO, pa = tmem + kColP + (n & 1) * 64;
            if (leader && !*abort_flag) {
#pragma unroll
                for (int kb = 0; kb < kBN / 16; ++kb)
                    mma_ts(d, pa + kb * 8, desc(lo_v + kb * (2048 >> 4)), idesc_pv, (n > 0 || kb > 0));
            }
            if (leader) {
                mma_commit(smem_u32(&bar->empty[seq % kSlots]));
                mma_commit(smem_u32(&bar->pv_done));
                if (n + 1 == n_tiles) mma_commit(smem_u32(&bar->o_final));
            }
            __syncwarp();
            // (issued behind PV(n): when S(n+2) lands, PV(n) has read P(n & 1), which softmax(n+2)
            // overwrites)
            if (n + 2 < n_tiles) qk(n + 2);
        }
    } else {
        // ------------------------------ softmax ------------------------------
        const int w = warp;                       // column quarter = TMEM lane quadrant
        const bool mine = lane < G;               // lanes with a query head
        const uint32_t lane_base = tmem + ((uint32_t)(w * 32) << 16);
        // this warp's copy of the G query rows: tile rows 32w .. 32w + G - 1 (16 lanes per row)
        {
            const int c = lane & 15, sub = lane >> 4;
            for (int r0 = 0; r0 < G; r0 += 2) {
                const int r = r0 + sub;
                if (r < G) {
                    const int row = w * 32 + r;
                    cp_async16(sQ + row * 128 + (c >> 3) * kHalfBytes + (((c & 7) ^ (row & 7)) << 4),
                               q + ((long long)b * Hq + h0 + r) * HD + c * 8, c < HD / 8 ? 16u : 0u);
                }
            }
            cp_async_commit();
        }
        // P = 0 outside this warp's own quarter, once for both buffers
        {
            uint32_t z16[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) z16[e] = 0u;
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) tmem_st16(lane_base + kColP + cc * 16, z16);
            tmem_wait_st();
        }
        cp_async_wait<0>();
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(smem_u32(&bar->q_full));

        float m = -INFINITY, l = 0.f;
        const uint32_t tO = lane_base + kColO;
        for (int n = 0; n < n_tiles; ++n) {
            const int bsel = n & 1;
            mbar_wait(smem_u32(&bar->s_full[bsel]), (n >> 1) & 1, abort_flag);
            tc_fence_after();
            uint32_t sr[32];
            tmem_ld32(lane_base + kColS + bsel * 128 + w * 32, sr);
            const uint32_t ok = bar->valid[n & 7][w];     // keys of this quarter that count
            tmem_wait_ld();
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int e = 0; e < 32; ++e)
                mx4[e & 3] = fmaxf(mx4[e & 3], ((ok >> e) & 1u) ? __uint_as_float(sr[e]) : -INFINITY);
            const float m_tile = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
            // the running max moves (and O is rescaled) only when a tile's max outgrew it by more
            // than the threshold: P stays inside the storage type's range
            float alpha = 1.f;
            const bool grow = mine && (m_tile > m + (kHalf ? kRescaleHalf : kRescaleBf16));
            if (grow) {
                alpha = ex2(m - m_tile);
                m = m_tile;
            }
            if (__any_sync(0xffffffffu, grow) && n > 0) {
                // O is complete through tile n-1 once PV(n-1) is: its commit is phase n-1 of
                // pv_done (PV(n) cannot have been issued yet, it waits for this tile's P)
                mbar_wait(smem_u32(&bar->pv_done), (n - 1) & 1, abort_flag);
                tc_fence_after();
#pragma unroll 1
                for (int cc = 0; cc < HD / 32; ++cc) {
                    uint32_t r[32];
                    tmem_ld32(tO + cc * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                    tmem_st32(tO + cc * 32, r);
                }
            }
            const float neg_m = (m == -INFINITY) ? 0.f : -m;
            float ps4[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t p16[16];
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                const float p0 = ((ok >> e) & 1u) ? ex2(fmaf(__uint_as_float(sr[e]), scale_log2, neg_m)) : 0.f;
                const float p1 = ((ok >> (e + 1)) & 1u) ? ex2(fmaf(__uint_as_float(sr[e + 1]), scale_log2, neg_m)) : 0.f;
                ps4[(e >> 1) & 3] += p0 + p1;
                p16[e >> 1] = pack16<kHalf>(p0, p1);
            }
            l = l * alpha + ((ps4[0] + ps4[1]) + (ps4[2] + ps4[3]));
            tmem_st16(lane_base + kColP + bsel * 64 + w * 16, p16);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(smem_u32(&bar->p_full[bsel]));
        }
        // ---- the four quarters of every head are merged through shared memory ----
        // (a barrier of its own for the end: pv_done may by now be one or two phases further, and
        // a wait on the parity of a phase two back would never return)
        mbar_wait(smem_u32(&bar->o_final), 0, abort_flag);
        tc_fence_after();
        // (every load of the ring has landed and every MMA that read it is complete)
        DtMerge *mg = reinterpret_cast<DtMerge *>(gen + kTileBytes);
        if (mine) {
            mg->m[w][lane] = m;
            mg->l[w][lane] = l;
        }
#pragma unroll 1
        for (int cc = 0; cc < HD / 32; ++cc) {
            uint32_t r[32];
            tmem_ld32(tO + cc * 32, r);
            tmem_wait_ld();
            if (mine) {
#pragma unroll
                for (int e = 0; e < 32; ++e) mg->o[w][lane][cc * 32 + e] = __uint_as_float(r[e]);
            }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        // thread = channel; the quarters are added in ascending order
        const int ch = threadIdx.x;
        for (int hh = 0; hh < G; ++hh) {
            float M = -INFINITY;
#pragma unroll
            for (int x = 0; x < 4; ++x) M = fmaxf(M, mg->m[x][hh]);
            float Ls = 0.f, Os = 0.f;
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float mr = mg->m[x][hh];
                if (mr != -INFINITY) {
                    const float wgt = ex2(mr - M);
                    Ls += mg->l[x][hh] * wgt;
                    Os += mg->o[x][hh][ch < HD ? ch : 0] * wgt;
                }
            }
            float *dst = ws + (((long long)b * Hq + h0 + hh) * n_chunks + blockIdx.x) * (HD + 2);
            if (ch < HD) dst[2 + ch] = Os;
            if (ch == 0) { dst[0] = M; dst[1] = Ls; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(status_word, ZIPVL_DEV_TIMEOUT);
    if (warp == kIssuerWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemColsDt);
    }
}

}  // namespace

bool decode_tc_supported(const zipvl_decode_desc &d) {
    if (d.n_kv_heads < 1 || d.n_q_heads % d.n_kv_heads) return false;
    const int G = d.n_q_heads / d.n_kv_heads;
    return (d.dtype == ZIPVL_BF16 || d.dtype == ZIPVL_F16) && (d.head_dim == 128 || d.head_dim == 96 || d.head_dim == 64) && G >= 2 && G <= kMaxGroup;
}

zipvl_status launch_decode_tc(const zipvl_decode_desc &d, float scale_log2, const void *q,
                              const void *k_new, const void *v_new, void *k_cache, void *v_cache,
                              const int64_t *cache_off, PageArgs pg, const int32_t *capacity,
                              int32_t *seq_lens, int max_len, int min_chunk, float *partials, int *lens,
                              int32_t *status_word, cudaStream_t st, int *chunk_out) {
    const int B = d.batch, Hq = d.n_q_heads, Hkv = d.n_kv_heads;
    // Rows per CTA: whole 128-row tiles, about two CTAs per SM over the batch, at most 16 tiles,
    // and never fewer rows than the chunk the workspace was sized for (min_chunk).
    const long long tiles = (long long)B * Hkv * ((max_len + kBN - 1) / kBN);
    long long tpc = (tiles + 295) / 296;
    if (tpc < 1) tpc = 1;
    if (tpc > kMaxTilesPerChunk) tpc = kMaxTilesPerChunk;
    int chunk = (int)tpc * kBN;
    if (chunk < min_chunk) chunk = ((min_chunk + kBN - 1) / kBN) * kBN;
    const int n_chunks = (max_len + chunk - 1) / chunk;
    *chunk_out = chunk;
    cudaError_t e = cudaSuccess;
#define ZIPVL_DT(H_, P_)                                                                            \
    {                                                                                               \
        auto kernel = decode_tc_kernel<H_, P_, 128>;                                                \
        if (d.head_dim == 96) kernel = decode_tc_kernel<H_, P_, 96>;                                \
        if (d.head_dim == 64) kernel = decode_tc_kernel<H_, P_, 64>;                                                     \
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDtSmem); \
        if (e == cudaSuccess)                                                                       \
            e = launch_dependent(kernel, dim3(n_chunks, Hkv, B), dim3(kThreadsDt), kDtSmem, st, Hq, Hkv, \
                                 scale_log2, (const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k_new, \
                                 (const __nv_bfloat16 *)v_new, (__nv_bfloat16 *)k_cache,            \
                                 (__nv_bfloat16 *)v_cache, cache_off, pg, capacity, seq_lens, max_len, \
                                 chunk, n_chunks, partials, lens, status_word);                     \
    }
    const bool half = d.dtype == ZIPVL_F16;
    if (half && pg.table) ZIPVL_DT(true, true)
    else if (half) ZIPVL_DT(true, false)
    else if (pg.table) ZIPVL_DT(false, true)
    else ZIPVL_DT(false, false)
#undef ZIPVL_DT
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "zipvl_decode: launch: %s", cudaGetErrorString(e));
    count_launches(1);
    return ZIPVL_OK;
}

}  // namespace zipvl
