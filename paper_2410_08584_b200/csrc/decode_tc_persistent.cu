// Grouped-query decode over the kept cache on the 5th-generation tensor cores: the persistent
// kernel for large batches (decode_tc.cu holds the one for small ones).
// (Algorithm 2; Eq. 4 append, Eq. 5 attention of one query token over the whole cache).
// 16-bit storage, head_dim 64, 96 or 128, 2 to 32 query heads per key/value head.
//
// With G query heads sharing one cached row, the CUDA-core kernel needs 2*G multiply-adds per
// cached element; from G = 3 on that, not HBM, sets its pace.  Here the G query rows of a kv head
// are rows of an MMA tile, so every cached byte is still read once and the arithmetic moves to
// the tensor pipe.
//
// Work = the key/value tiles (128 cache rows of one kv head) of all requests, in the order
// request, kv head, tile.  The launch is persistent: one CTA per SM, CTA i takes tiles
// [i*q, (i+1)*q) of that sequence, q the same for all (every CTA computes the lengths' prefix
// sums itself; no counter, nothing to clear).  A CTA's range is cut into SEGMENTS at the
// (request, kv head) boundaries; a segment yields one partial (m, l, o[128]) per query head,
// which the merge kernel of the CUDA-core path combines.
//   warps 0-3  softmax.  The tile has 128 rows and only G are needed, so the G query rows are
//              loaded FOUR times: warp w (which owns TMEM lanes 32w..32w+31) has its copy at rows
//              32w + o .. 32w + o + G - 1, takes the keys 32w..32w+31 of every tile and leaves
//              P = 0 for the others, so the four warps (one per scheduler and exp2 unit) share a
//              tile's columns and each keeps its own running (max, sum) and its own rows of O: a
//              segment leaves four partials per query head.  With G <= 16 the offset o alternates
//              between 0 and 16 from segment to segment, so the next segment's query rows are in
//              place (and its first scores computed) before this one ends.  Rows nobody owns hold
//              whatever they hold: a row of an MMA result depends on its own row of A only.
//   warps 4-15 producers, in groups of four warps (one group fills one tile, a warp per 32 rows):
//              16 lanes copy one cached row (256 B) with 16-byte async copies into the
//              128-byte-swizzled tile; K and V tiles go through one ring of six 32 KB slots that
//              runs on across segments, so the loads never drain between work items.  Rows
//              behind the request's length are zero-filled and flagged (one bit per row).  The
//              appended row (Eq. 4) is taken from k_new / v_new and stored into the cache.
//   warp 16    issues tcgen05.mma: S = Q K^T (shared-memory operands) into one of two S buffers,
//              O = / += P V (P from tensor memory, V as MN-major operand); the first PV of a
//              segment overwrites O.
// Tensor memory (512 columns): S0 | S1 | P0 P1 (64 each) | O.  Every wait is bounded.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace zipvl {
namespace {

using namespace ptx;

constexpr int kBN = 128;
constexpr int kSlots = 6;              // ring of K / V tiles (K0 V0 K1 V1 K2 V2)
// A warp can only have so many 16-byte async copies outstanding, so the bytes in flight -- and
// with them the bandwidth the SM can draw -- grow with the number of producer warps, not with the
// depth of one warp's queue: four warps alone stay near 11 bytes per clock.  Group j takes the
// tiles j, j + kGroups, ... of the ring sequence K0 V0 K1 V1 ...
constexpr int kGroups = 3;
// (every use of a ring slot must fall to the same group, which fills its tiles in order: a
// slot's "empty" barrier is then never more than one phase behind its reader)
static_assert(kSlots % kGroups == 0, "a group owns whole ring slots");
constexpr int kWindow = 3;             // tile loads in flight per producer thread
// warps: softmax 0-3, the producers, the issuer.  96 registers per thread: the CTA then leaves room
// on its SM for the CTAs of the merge kernel, which are launched as programmatic dependents and
// wait there until this kernel is done (a launch that fills the register file keeps them out, and
// every step pays the merge's launch latency)
constexpr int kSoftmaxWarps = 4;
constexpr int kFirstProducer = 4;
constexpr int kIssuerWarp = kFirstProducer + 4 * kGroups;
constexpr int kHalfBytes = 128 * 128;
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kThreadsDt = 32 * (kIssuerWarp + 1);
// (the bound the compiler sees: 640 threads per CTA cap a thread at 96 registers; 544 are launched)
constexpr int kBoundThreadsDt = 640;
constexpr uint32_t kTmemColsDt = 512;
constexpr uint32_t kColS = 0, kColP = 256, kColO = 384;
constexpr int kMaxGroup = 32;       // query heads per kv head: one warp's 32 rows of the tile
constexpr float kRescaleBf16 = 32.0f, kRescaleHalf = 8.0f;   // octaves the running max may lag

struct DtBarriers {
    uint64_t q_full[2];                // the query rows of a segment are in place (per row set)
    uint64_t full[kSlots];
    uint64_t empty[kSlots];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t pv_done;                  // once per tile, behind PV(n)
    uint64_t seg_pv;                   // behind the last PV of a segment
    uint32_t tmem_base;
    int abort_flag;
    uint32_t valid[8][4];              // per key tile (mod 8) and 32-row block: rows that count
    long long scan_total[kThreadsDt / 32];
    int start_b;                       // request that holds the CTA's first tile ...
    long long start_R;                 // ... and the tiles (per kv head) of the requests before it
};

constexpr size_t kDtSmem = kTileBytes * (1 + kSlots) + sizeof(DtBarriers) + 1024;

struct DtArgs {
    int B, Hq, Hkv, max_len, n_slots, q_min;
    float scale_log2;
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *k_cache, *v_cache;
    const int64_t *cache_off;
    PageArgs pg;
    const int32_t *capacity;
    int32_t *seq_lens;
    float *ws;                         // partials: [B][Hq][n_slots][head_dim + 2]
    int *lens;                         // (length, appended) per request, for the merge
    int *used;                         // slots in use per (request, kv head), for the merge
    int32_t *status_word;
};

// What a step does with request b: the length it attends over and the row it appends (-1: none).
struct Req {
    int len, new_row;
    long long coff;
    unsigned flags;                    // device-status bits this request raises
};
template <bool kPaged>
__device__ __forceinline__ Req request(const DtArgs &a, int b) {
    Req r;
    const int old_len = a.seq_lens[b];
    const int cap = a.capacity[b];
    r.coff = kPaged ? 0ll : a.cache_off[b];
    r.flags = 0;
    // a length that is negative or beyond the capacity, or a cache offset that breaks the 16-byte
    // alignment of the row copies: the request is skipped as a whole and reported
    const bool bad = old_len < 0 || old_len > cap || ((r.coff * 2) & 15) != 0;
    if (bad) r.flags |= ZIPVL_DEV_BAD_INDEX;
    const bool appended = !bad && a.k_new != nullptr && old_len < cap;
    if (a.k_new != nullptr && !bad && !appended) r.flags |= ZIPVL_DEV_CAPACITY;
    r.len = bad ? 0 : old_len + (appended ? 1 : 0);
    if (r.len > a.max_len) {
        r.flags |= ZIPVL_DEV_CAPACITY;
        r.len = a.max_len;
    }
    r.new_row = appended ? old_len : -1;
    return r;
}
__device__ __forceinline__ int tiles_of(int len) { return (len + kBN - 1) / kBN; }

// A position in the tile sequence: tile t of kv head g of request b (nt tiles per kv head, R tiles
// per kv head in the requests before it), and how many (request, kv head) boundaries were crossed.
template <bool kPaged>
struct Walker {
    int b, g, t, nt, seg;
    long long R;
    Req r;
    __device__ __forceinline__ void start(const DtArgs &a, int b0, long long R0, long long pos) {
        b = b0; R = R0; seg = 0;
        r = request<kPaged>(a, b);
        nt = tiles_of(r.len);
        const long long rem = pos - (long long)a.Hkv * R;      // (nt > 0 by the choice of b0)
        g = (int)(rem / nt);
        t = (int)(rem % nt);
    }
    // forward by d tiles (d >= 0); stays inside the sequence by the caller's bounds
    __device__ __forceinline__ void advance(const DtArgs &a, int d) {
        t += d;
        while (t >= nt) {
            t -= nt;
            ++seg;
            if (++g == a.Hkv) {
                g = 0;
                R += nt;
                do {
                    if (++b >= a.B) { b = a.B - 1; nt = 1 << 30; return; }   // (past the end: never used)
                    r = request<kPaged>(a, b);
                    nt = tiles_of(r.len);
                } while (nt == 0);
            }
        }
    }
    __device__ __forceinline__ long long pair_start(const DtArgs &a) const {
        return (long long)a.Hkv * R + (long long)g * nt;
    }
};

// HD: head_dim (64, 96 or 128); the shared-memory tiles stay 128 wide and the narrower heads use
// the front of them
template <bool kHalf, bool kPaged, int HD>
__global__ void __launch_bounds__(kBoundThreadsDt, 1)
decode_tcp_kernel(DtArgs a) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char *gen = smem_raw + (base - raw);
    const uint32_t sQ = base;
    const uint32_t sRing = base + kTileBytes;
    DtBarriers *bar = reinterpret_cast<DtBarriers *>(gen + kTileBytes * (1 + kSlots));
    volatile int *abort_flag = &bar->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = a.Hq / a.Hkv;

    grid_launch_dependents();
    // lengths and caches may be the previous kernel's output
    grid_dependency_wait(a.q, a.k_new, a.v_new, a.k_cache, a.v_cache, a.cache_off, a.capacity, a.seq_lens,
                         a.pg.table);

    // ---- every CTA sums the tiles of all requests: its own range follows from the total ----
    // thread i takes a contiguous block of requests; CTA 0 also leaves what the merge kernel
    // needs (the step's length, "appended", no partials for an empty request) and reports
    const int per = (a.B + kThreadsDt - 1) / kThreadsDt;
    const int b_lo = min(a.B, (int)threadIdx.x * per), b_hi = min(a.B, b_lo + per);
    long long mine = 0;
    for (int b = b_lo; b < b_hi; ++b) {
        const Req r = request<kPaged>(a, b);
        mine += tiles_of(r.len);
        if (blockIdx.x == 0) {
            if (r.flags) report(a.status_word, r.flags);
            a.lens[2 * b] = r.len;
            a.lens[2 * b + 1] = r.new_row >= 0 ? 1 : 0;
            if (r.len == 0)
                for (int g = 0; g < a.Hkv; ++g) a.used[b * a.Hkv + g] = 0;
        }
    }
    long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const long long v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) bar->scan_total[warp] = incl;
    __syncthreads();
    long long before = 0, per_head = 0;
#pragma unroll
    for (int w = 0; w < kThreadsDt / 32; ++w) {
        const long long v = bar->scan_total[w];
        if (w < warp) before += v;
        per_head += v;
    }
    before += incl - mine;                         // tiles per kv head in front of this thread's block
    const long long total = per_head * a.Hkv;
    long long q = (total + gridDim.x - 1) / gridDim.x;
    if (q < a.q_min) q = a.q_min;
    const long long lo = (long long)blockIdx.x * q;
    if (lo >= total) return;                       // (also: nothing cached anywhere)
    const long long hi = lo + q < total ? lo + q : total;
    const int n_tiles = (int)(hi - lo);
    if (mine > 0 && before * a.Hkv <= lo && lo < (before + mine) * a.Hkv) {
        // the request that holds tile lo is in this thread's block
        long long R = before;
        for (int b = b_lo; b < b_hi; ++b) {
            const long long nt = tiles_of(request<kPaged>(a, b).len);
            if (lo < (R + nt) * a.Hkv) { bar->start_b = b; bar->start_R = R; break; }
            R += nt;
        }
    }
    if (threadIdx.x == 0) {
        for (int x = 0; x < 2; ++x) {
            mbar_init(smem_u32(&bar->q_full[x]), 32 * kSoftmaxWarps);
            mbar_init(smem_u32(&bar->s_full[x]), 1);
            mbar_init(smem_u32(&bar->p_full[x]), 32 * kSoftmaxWarps);
        }
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&bar->full[s]), 128);
            mbar_init(smem_u32(&bar->empty[s]), 1);
        }
        mbar_init(smem_u32(&bar->pv_done), 1);
        mbar_init(smem_u32(&bar->seg_pv), 1);
        bar->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == kIssuerWarp) tmem_alloc(smem_u32(&bar->tmem_base), kTmemColsDt);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bar->tmem_base;
    const long long row_pitch = (long long)a.Hkv * HD;          // elements between cache rows
    Walker<kPaged> wk;
    wk.start(a, bar->start_b, bar->start_R, lo);

    // query rows of even and odd segments in different lanes (rows) where the group is small enough
    const bool two_sets = G <= 16;
    if (warp >= kFirstProducer && warp < kIssuerWarp) {
        // ------------------------------ producers ------------------------------
        const int p = (warp - kFirstProducer) & 3;       // this warp's 32 rows of every 128-row tile
        const int group = (warp - kFirstProducer) >> 2;
        const int c = lane & 15, sub = lane >> 4;
        const int total_seq = 2 * n_tiles;               // K0 V0 K1 V1 ...
        // this group's share of the sequence: seq = group + j * kGroups
        const int mine_n = group < total_seq ? (total_seq - group + kGroups - 1) / kGroups : 0;
        int at = 0;                                      // tile (of this CTA) the walker stands on
        auto issue = [&](int seq) {
            const int n = seq >> 1, kind = seq & 1;
            wk.advance(a, n - at);
            at = n;
            const int j0 = wk.t * kBN;                   // first cache row of the tile
            const int32_t *my_table = kPaged ? a.pg.table + (long long)wk.b * a.pg.stride : nullptr;
            const long long head_off = wk.r.coff + (long long)wk.g * HD;
            // one lane per row: where the row lives (-1: behind the length, or in a page outside
            // the pool, which is reported and left out of the attention)
            long long my_off = -1;
            {
                const int row = j0 + p * 32 + lane;
                if (row < wk.r.len) {
                    if (!kPaged) {
                        my_off = row * row_pitch;
                    } else {
                        const int page = my_table[row >> a.pg.shift];
                        if (page < 0 || page >= a.pg.n_pages) { if (kind == 0) report(a.status_word, ZIPVL_DEV_BAD_INDEX); }
                        else my_off = (((long long)page << a.pg.shift) + (row & ((1 << a.pg.shift) - 1))) * row_pitch;
                    }
                }
                const uint32_t word = __ballot_sync(0xffffffffu, my_off >= 0);
                if (lane == 0 && kind == 0) bar->valid[n & 7][p] = word;
            }
            const uint32_t tile = sRing + (seq % kSlots) * kTileBytes;
            __nv_bfloat16 *cache = kind ? a.v_cache : a.k_cache;
            const __nv_bfloat16 *fresh = (kind ? a.v_new : a.k_new);
            if (fresh) fresh += ((long long)wk.b * a.Hkv + wk.g) * HD;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int r = p * 32 + i + 16 * sub;                    // row of the tile
                const long long off = __shfl_sync(0xffffffffu, my_off, i + 16 * sub);
                const uint32_t dst = tile + r * 128 + (c >> 3) * kHalfBytes + (((c & 7) ^ (r & 7)) << 4);
                const bool ok = off >= 0;
                const bool piece = c < HD / 8;                          // (a row has HD / 8 chunks of 16 bytes)
                const __nv_bfloat16 *src = cache + (ok ? off : 0) + head_off + (piece ? c : 0) * 8;
                if (ok && j0 + r == wk.r.new_row) {
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
    } else if (warp >= kIssuerWarp) {
        // ------------------------------ MMA issuer ------------------------------
        if (warp == kIssuerWarp) {
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
        // Two positions in the CTA's tiles: the PV of tile n and the QK two tiles ahead, each with
        // its segment's ordinal and whether the tile opens / closes its segment.
        auto opens = [&](const Walker<kPaged> &w, int n) { return n == 0 || w.t == 0; };
        auto closes = [&](const Walker<kPaged> &w, int n) { return n == n_tiles - 1 || w.t == w.nt - 1; };
        Walker<kPaged> wq = wk, wp = wk;              // wq: next QK, wp: next PV
        int nq = 0;
        // S(n) = Q K(n)^T into buffer n & 1; the commits free K's slot and announce S
        auto qk = [&]() {
            const int n = nq;
            if (opens(wq, n)) {
                // the segment's query rows (the softmax warps put them into the Q tile): row set
                // seg & 1 in its (seg / 2)-th use, or the one set in its seg-th
                const int set = two_sets ? (wq.seg & 1) : 0, use = two_sets ? (wq.seg >> 1) : wq.seg;
                mbar_wait(smem_u32(&bar->q_full[set]), use & 1, abort_flag);
            }
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
            wq.advance(a, 1);
            ++nq;
        };
        qk();
        if (n_tiles > 1) qk();
        for (int n = 0; n < n_tiles; ++n) {
            // P(n) is written: softmax(n) is also done reading S(n), so QK(n+2) may reuse it.  At a
            // segment's first tile the softmax warps have read the rows of O of the segment before
            // (they do that before they turn to this tile), so this PV may overwrite O.
            mbar_wait(smem_u32(&bar->p_full[n & 1]), (n >> 1) & 1, abort_flag);
            const bool first = opens(wp, n), last = closes(wp, n);
            const int seq = 2 * n + 1;
            wait_full(seq);
            const uint32_t lo_v = (lo_ring + (seq % kSlots) * (kTileBytes >> 4)) |
                                  ((uint32_t)(kHalfBytes >> 4) << 16);
            const uint32_t d = tmem + kColO, pa = tmem + kColP + (n & 1) * 64;
            if (leader && !*abort_flag) {
#pragma unroll
                for (int kb = 0; kb < kBN / 16; ++kb)
                    mma_ts(d, pa + kb * 8, desc(lo_v + kb * (2048 >> 4)), idesc_pv, (!first || kb > 0));
            }
            if (leader) {
                mma_commit(smem_u32(&bar->empty[seq % kSlots]));
                mma_commit(smem_u32(&bar->pv_done));
                if (last) mma_commit(smem_u32(&bar->seg_pv));
            }
            __syncwarp();
            wp.advance(a, 1);
            // (issued behind PV(n): when S(n+2) lands, PV(n) has read P(n & 1), which softmax(n+2)
            // overwrites)
            if (nq < n_tiles) qk();
        }
        }
    } else {
        // ------------------------------ softmax (warps 0-3) ------------------------------
        const int w = warp;                       // column quarter = TMEM lane quadrant
        const uint32_t lane_base = tmem + ((uint32_t)(w * 32) << 16);
        const uint32_t tO = lane_base + kColO;
        // this warp's copy of a segment's G query rows: tile rows 32w + o .. 32w + o + G - 1
        // (16 lanes per row); every lane of the four warps arrives
        auto load_q = [&](int b, int g, int o, int set) {
            const int c = lane & 15, sub = lane >> 4;
            for (int r0 = 0; r0 < G; r0 += 2) {
                const int r = r0 + sub;
                if (r < G) {
                    const int row = w * 32 + o + r;
                    cp_async16(sQ + row * 128 + (c >> 3) * kHalfBytes + (((c & 7) ^ (row & 7)) << 4),
                               a.q + ((long long)b * a.Hq + g * G + r) * HD + c * 8, c < HD / 8 ? 16u : 0u);
                }
            }
            cp_async_commit();
            cp_async_wait<0>();
            fence_proxy_async();
            mbar_arrive(smem_u32(&bar->q_full[set]));
        };
        // P = 0 outside this warp's own quarter of the keys, once for both buffers: no one ever
        // writes those columns of this warp's lanes
        {
            uint32_t z16[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) z16[e] = 0u;
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) tmem_st16(lane_base + kColP + cc * 16, z16);
            tmem_wait_st();
            tc_fence_before();
        }
        load_q(wk.b, wk.g, 0, 0);
        int n = 0;
        while (n < n_tiles) {
            const int cnt = min(wk.nt - wk.t, n_tiles - n);      // tiles of this segment in the CTA
            const int seg = wk.seg;
            const int off = two_sets ? 16 * (seg & 1) : 0;       // this segment's lanes
            const bool mine = lane >= off && lane < off + G;      // lanes with a query head
            const bool more = n + cnt < n_tiles;                  // another segment follows
            Walker<kPaged> nx = wk;
            if (more) nx.advance(a, cnt);
            // the next segment's query rows go to the other row set right away: the MMAs of the
            // segment that used it last are complete (its O was read behind them)
            if (more && two_sets) load_q(nx.b, nx.g, 16 * ((seg + 1) & 1), (seg + 1) & 1);
            float m = -INFINITY, l = 0.f;
            for (int i = 0; i < cnt; ++i) {
                const int nn = n + i, bsel = nn & 1;
                mbar_wait(smem_u32(&bar->s_full[bsel]), (nn >> 1) & 1, abort_flag);
                tc_fence_after();
                // one row set only: every QK of this segment is complete once its last S is here,
                // so the next segment's query rows may replace this one's
                if (more && !two_sets && i == cnt - 1) load_q(nx.b, nx.g, 0, 0);
                uint32_t sr[32];
                tmem_ld32(lane_base + kColS + bsel * 128 + w * 32, sr);
                const uint32_t ok = bar->valid[nn & 7][w];     // keys of this quarter that count
                tmem_wait_ld();
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    mx4[e & 3] = fmaxf(mx4[e & 3], ((ok >> e) & 1u) ? __uint_as_float(sr[e]) : -INFINITY);
                const float m_tile = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;
                // the running max moves (and O is rescaled) only when a tile's max outgrew it by more
                // than the threshold: P stays inside the storage type's range
                float alpha = 1.f;
                const bool grow = mine && (m_tile > m + (kHalf ? kRescaleHalf : kRescaleBf16));
                if (grow) {
                    alpha = ex2(m - m_tile);
                    m = m_tile;
                }
                if (__any_sync(0xffffffffu, grow) && i > 0) {
                    // O is complete through tile nn-1 once PV(nn-1) is: its commit is phase nn-1 of
                    // pv_done (S(nn) landed behind PV(nn-2), so the barrier is in phase nn-1 or nn:
                    // the parity is unambiguous; PV(nn) waits for this tile's P)
                    mbar_wait(smem_u32(&bar->pv_done), (nn - 1) & 1, abort_flag);
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
                    const float p0 = ((ok >> e) & 1u) ? ex2(fmaf(__uint_as_float(sr[e]), a.scale_log2, neg_m)) : 0.f;
                    const float p1 = ((ok >> (e + 1)) & 1u) ? ex2(fmaf(__uint_as_float(sr[e + 1]), a.scale_log2, neg_m)) : 0.f;
                    ps4[(e >> 1) & 3] += p0 + p1;
                    p16[e >> 1] = pack16<kHalf>(p0, p1);
                }
                l = l * alpha + ((ps4[0] + ps4[1]) + (ps4[2] + ps4[3]));
                tmem_st16(lane_base + kColP + bsel * 64 + w * 16, p16);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&bar->p_full[bsel]));
            }
            // ---- the segment's partials: (m, l, o[128]) of this quarter of the keys, per query head ----
            mbar_wait(smem_u32(&bar->seg_pv), seg & 1, abort_flag);
            tc_fence_after();
            const long long pair0 = wk.pair_start(a);
            const int first_cta = (int)(pair0 / q);
            const int slot = kSoftmaxWarps * ((int)blockIdx.x - first_cta) + w;
            float *dst = a.ws + (((long long)wk.b * a.Hq + wk.g * G + (lane - off)) * a.n_slots + slot) * (HD + 2);
            if (mine) {
                dst[0] = m;
                dst[1] = l;
            }
#pragma unroll 1
            for (int cc = 0; cc < HD / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(tO + cc * 32, r);
                tmem_wait_ld();
                if (mine) {
#pragma unroll
                    for (int e = 0; e < 32; e += 2)
                        *reinterpret_cast<float2 *>(dst + 2 + cc * 32 + e) =
                            make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1]));
                }
            }
            tc_fence_before();
            // the CTA that holds a pair's first tile says how many slots the pair fills
            if (wk.t == 0 && w == 0 && lane == 0)
                a.used[wk.b * a.Hkv + wk.g] = kSoftmaxWarps * ((int)((pair0 + wk.nt - 1) / q) - first_cta + 1);
            n += cnt;
            wk.advance(a, cnt);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) report(a.status_word, ZIPVL_DEV_TIMEOUT);
    if (warp == kIssuerWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemColsDt);
    }
}

}  // namespace

zipvl_status launch_decode_tcp(const zipvl_decode_desc &d, float scale_log2, const void *q,
                              const void *k_new, const void *v_new, void *k_cache, void *v_cache,
                              const int64_t *cache_off, PageArgs pg, const int32_t *capacity,
                              int32_t *seq_lens, int max_len, int n_slots, float *partials, int *lens,
                              int *used, int32_t *status_word, cudaStream_t st) {
    if (!decode_tc_supported(d) || d.n_q_heads / d.n_kv_heads > kMaxGroup)
        return fail(ZIPVL_ERR_UNSUPPORTED, "zipvl_decode: this shape does not run on the tensor-core kernel");
    static int n_sm_of[64] = {0};                  // multiprocessors per device, asked once
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !n_sm_of[dev])
        cudaDeviceGetAttribute(&n_sm_of[dev], cudaDevAttrMultiProcessorCount, dev);
    const int n_sm = (dev >= 0 && dev < 64 && n_sm_of[dev] > 0) ? n_sm_of[dev] : 148;
    DtArgs a;
    a.B = d.batch; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.max_len = max_len;
    a.n_slots = n_slots;
    // a (request, kv head) pair of t tiles is shared by at most ceil(t / q) + 1 CTAs, each of which
    // needs slots of its own: q may not fall below this, however few tiles there are in all
    // (n_slots counts partials: kSoftmaxWarps of them per CTA that shares a pair)
    const int nt_bound = (max_len + kBN - 1) / kBN;
    const int ctas_per_pair = n_slots / kSoftmaxWarps;
    a.q_min = ctas_per_pair > 1 ? (nt_bound + ctas_per_pair - 2) / (ctas_per_pair - 1) : nt_bound;
    a.scale_log2 = scale_log2;
    a.q = (const __nv_bfloat16 *)q; a.k_new = (const __nv_bfloat16 *)k_new; a.v_new = (const __nv_bfloat16 *)v_new;
    a.k_cache = (__nv_bfloat16 *)k_cache; a.v_cache = (__nv_bfloat16 *)v_cache;
    a.cache_off = cache_off; a.pg = pg; a.capacity = capacity; a.seq_lens = seq_lens;
    a.ws = partials; a.lens = lens; a.used = used; a.status_word = status_word;
    const int grid = n_sm;                         // persistent: one CTA per SM
    cudaError_t e = cudaSuccess;
#define ZIPVL_DT(H_, P_)                                                                            \
    {                                                                                               \
        auto kernel = decode_tcp_kernel<H_, P_, 128>;                                               \
        if (d.head_dim == 96) kernel = decode_tcp_kernel<H_, P_, 96>;                               \
        if (d.head_dim == 64) kernel = decode_tcp_kernel<H_, P_, 64>;                               \
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDtSmem); \
        if (e == cudaSuccess)                                                                       \
            e = launch_dependent(kernel, dim3(grid), dim3(kThreadsDt), kDtSmem, st, a);             \
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
