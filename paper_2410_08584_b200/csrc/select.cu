// Layer-adaptive budget (Eq. 7) and important-token set (Eq. 9).
//
// Nothing is sorted.  Both questions are threshold searches on the
// order-preserving bit pattern of a score, answered by a radix descent (12 bits,
// then 8, then either a direct comparison of the at most 128 tokens left or the
// last 12 bits):
//   budget   the largest score value v* such that the scores >= v* sum to at least
//            tau * S; p = #{a > v*} + the number of copies of v* still needed;
//   top-p    the p-th largest ranking score u*; ties at u* go to the smaller
//            position.
// Rows of up to 4096 tokens run on one CTA that holds the row in registers (see
// select_solo_kernel further down).  Longer rows: ceil(L / 1024) CTAs histogram 1024
// tokens each on the top 12 key bits (count and sum of the budget score, count of the
// ranking score), add their
// non-empty bins to a global histogram (64 KB of the workspace, cleared by a memset
// node in front of the kernel) and the last CTA to finish (ticket) goes on alone.
// That CTA finds the crossing bin (one warp scans the occupied bin range), refines
// inside it over the tokens that match the prefix, then writes T in ascending
// position with one block-wide prefix sum.  The two searches are two passes of one
// loop body.  Sums are 64-bit fixed point (2^-34 units, round to nearest), exact and
// order independent, so the result repeats bit for bit.
#include "common.cuh"

namespace zipvl {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kBins = 4096;                  // 12-bit digits
constexpr int kWarpBins = 16;                 // bins per lane when one warp scans a histogram
constexpr int kBatch = 3;                     // row values loaded ahead of use, per thread
constexpr int kSoloMax = 4096;               // sequences up to this length run on one CTA
constexpr double kFxScale = 17179869184.0;   // 2^34

__device__ __forceinline__ unsigned long long to_fx(float v) {
    return (v > 0.f) ? __double2ull_rn((double)v * kFxScale) : 0ull;
}

// global histogram in the workspace: [cnt_budget | cnt_rank | sum_lo | sum_hi | ticket]
struct GlobalHist {
    unsigned int cnt_b[kBins];
    unsigned int cnt_r[kBins];
    unsigned long long sum_b[kBins];
    unsigned int rng[4];      // occupied level-1 bins, see SelCtl::rng
    unsigned int ticket;
};

// shared memory of one CTA (dynamic): the same four arrays, 64-bit sums as two words
struct SelSmem {
    unsigned int cnt_b[kBins];
    unsigned int cnt_r[kBins];
    unsigned int sum_lo[kBins];
    unsigned int sum_hi[kBins];
};

struct SelCtl {                                // static shared memory
    unsigned long long scan64[32];
    unsigned int scan32[32];
    unsigned int scan32b[32];
    unsigned long long sum_gt, bin_sum;
    unsigned int hit, hit_bin, n_cand, cnt_gt, bin_cnt, is_last;
    // occupied level-1 bins as maxima (so zero means empty): budget {hi, 4095 - lo},
    // ranking {hi, 4095 - lo}
    unsigned int rng[4];
};

__device__ __forceinline__ unsigned long long bin_sum64(const SelSmem &sm, int b) {
    return ((unsigned long long)sm.sum_hi[b] << 32) | sm.sum_lo[b];
}

// 64-bit add into a lo/hi pair of shared-memory words with native 32-bit atomics
__device__ __forceinline__ void smem_add64(SelSmem &sm, int b, unsigned long long v) {
    const unsigned int lo = (unsigned int)v, hi = (unsigned int)(v >> 32);
    const unsigned int old = atomicAdd(&sm.sum_lo[b], lo);
    const unsigned int carry = (old + lo < old) ? 1u : 0u;
    if (hi | carry) atomicAdd(&sm.sum_hi[b], hi + carry);
}

// Histogram update for one element per lane.  When every active lane of the warp
// has the same digit (all-equal scores, the worst case for atomics) the warp adds
// once; otherwise each lane adds for itself.
__device__ __forceinline__ void hist_add(unsigned int *cnt, SelSmem *sums, bool active,
                                         unsigned int d, unsigned long long v,
                                         unsigned int *rng = nullptr) {
    const unsigned int amask = __ballot_sync(0xffffffffu, active);
    if (amask == 0) return;
    if (rng) {
        // one pair of atomics per warp keeps the range of occupied bins
        const unsigned int dmax = __reduce_max_sync(0xffffffffu, active ? d : 0u);
        const unsigned int imax = __reduce_max_sync(0xffffffffu, active ? (kBins - 1) - d : 0u);
        if ((threadIdx.x & 31) == 0) { atomicMax(&rng[0], dmax); atomicMax(&rng[1], imax); }
    }
    const int leader = __ffs(amask) - 1;
    const unsigned int d0 = __shfl_sync(0xffffffffu, d, leader);
    const bool same = __ballot_sync(0xffffffffu, active && d != d0) == 0;
    if (same) {
        unsigned long long s = 0;
        if (sums) {
            const unsigned int l0 = active ? (unsigned int)(v & 0x3fffffu) : 0u;
            const unsigned int l1 = active ? (unsigned int)((v >> 22) & 0x3fffffu) : 0u;
            const unsigned int l2 = active ? (unsigned int)(v >> 44) : 0u;
            s = (unsigned long long)__reduce_add_sync(0xffffffffu, l0) +
                ((unsigned long long)__reduce_add_sync(0xffffffffu, l1) << 22) +
                ((unsigned long long)__reduce_add_sync(0xffffffffu, l2) << 44);
        }
        if ((int)(threadIdx.x & 31) == leader) {
            atomicAdd(&cnt[d0], (unsigned int)__popc(amask));
            if (sums) smem_add64(*sums, d0, s);
        }
    } else if (active) {
        atomicAdd(&cnt[d], 1u);
        if (sums) smem_add64(*sums, d, v);
    }
}

// block-wide sum of a u64 (every thread returns the total); 32 warps, no serial loop
__device__ unsigned long long block_sum64(unsigned long long v, SelCtl &c) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) c.scan64[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long t = c.scan64[threadIdx.x & 31];
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    return t;
}

// block-wide exclusive prefix sums in thread order of a (u32, u64) pair: a shuffle
// scan inside each warp, then every warp scans the 32 warp totals again by shuffles
__device__ void block_excl_scan2(unsigned int vc, unsigned long long vs, SelCtl &c,
                                 unsigned int *pc, unsigned long long *ps) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned int ic = vc;
    unsigned long long is = vs;
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned int nc = __shfl_up_sync(0xffffffffu, ic, o);
        const unsigned long long ns = __shfl_up_sync(0xffffffffu, is, o);
        if (lane >= o) { ic += nc; is += ns; }
    }
    __syncthreads();
    if (lane == 31) { c.scan32[w] = ic; c.scan64[w] = is; }
    __syncthreads();
    const unsigned int tc = c.scan32[lane];
    const unsigned long long ts = c.scan64[lane];
    unsigned int wc = tc;
    unsigned long long ws = ts;
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned int nc = __shfl_up_sync(0xffffffffu, wc, o);
        const unsigned long long ns = __shfl_up_sync(0xffffffffu, ws, o);
        if (lane >= o) { wc += nc; ws += ns; }
    }
    const unsigned int bc = __shfl_sync(0xffffffffu, wc - tc, w);
    const unsigned long long bs = __shfl_sync(0xffffffffu, ws - ts, w);
    *pc = bc + ic - vc;
    *ps = bs + is - vs;
}

// Scan n_bins (<= 4096) bins from the top.  by_sum: first non-empty bin at which
// carry_sum + descending cumulative SUM >= target; else first bin at which
// carry_cnt + descending cumulative COUNT >= target.  Publishes in c: hit (0xffffffff
// when no bin qualifies) and hit_bin, cnt_gt / sum_gt (everything above the bin, carries included) and the
// bin's own count / sum.  All threads call; results valid after return.
__device__ void find_bin(const unsigned int *cnt, const SelSmem *sums, int n_bins, bool by_sum,
                         unsigned long long target, unsigned int carry_cnt,
                         unsigned long long carry_sum, SelCtl &c, int lo = 0, int hi = -1) {
    if (hi < lo) { lo = 0; hi = n_bins - 1; }          // no range given: all bins
    if (hi - lo + 1 <= 32 * kWarpBins) {
        // Few occupied bins (scores span a few dozen octaves at most): one warp scans
        // them, kWarpBins per lane from the top, with a shuffle scan in between.
        __syncthreads();
        if (threadIdx.x < 32) {
            const int lane = threadIdx.x;
            const int per = (hi - lo + 1 + 31) / 32;
            unsigned int lc = 0;
            unsigned long long ls = 0;
            for (int i = 0; i < per; ++i) {
                const int b = hi - (lane * per + i);
                if (b >= lo) {
                    lc += cnt[b];
                    if (sums) ls += bin_sum64(*sums, b);
                }
            }
            unsigned int ic = lc;
            unsigned long long is = ls;
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int nc = __shfl_up_sync(0xffffffffu, ic, o);
                const unsigned long long ns = __shfl_up_sync(0xffffffffu, is, o);
                if (lane >= o) { ic += nc; is += ns; }
            }
            unsigned int run_c = carry_cnt + ic - lc;
            unsigned long long run_s = carry_sum + is - ls;
            int my_hit = -1;
            unsigned int bc = 0;
            unsigned long long bs = 0;
            for (int i = 0; i < per && my_hit < 0; ++i) {
                const int b = hi - (lane * per + i);
                if (b < lo) break;
                const unsigned int cb = cnt[b];
                const unsigned long long sb = sums ? bin_sum64(*sums, b) : 0ull;
                const bool ok = cb > 0 && (by_sum ? (run_s + sb >= target)
                                                  : ((unsigned long long)run_c + cb >= target));
                if (ok) { my_hit = b; bc = cb; bs = sb; }
                else { run_c += cb; run_s += sb; }
            }
            const unsigned int hits = __ballot_sync(0xffffffffu, my_hit >= 0);
            if (hits == 0) {
                if (lane == 0) c.hit = 0xffffffffu;
            } else if (lane == __ffs(hits) - 1) {      // lowest lane = highest bins
                c.hit = 0;
                c.hit_bin = (unsigned int)my_hit;
                c.cnt_gt = run_c;
                c.sum_gt = run_s;
                c.bin_cnt = bc;
                c.bin_sum = bs;
            }
        }
        __syncthreads();
        return;
    }
    const int per = n_bins / kSelThreads;              // 4 (4096 bins) or 0 (256 bins)
    const int nb = per > 0 ? per : 1;
    const bool mine = per > 0 || (int)threadIdx.x < n_bins;
    unsigned int lc = 0;
    unsigned long long ls = 0;
    if (mine) {
        for (int i = 0; i < nb; ++i) {
            const int b = n_bins - 1 - ((int)threadIdx.x * nb + i);
            lc += cnt[b];
            if (sums) ls += bin_sum64(*sums, b);
        }
    }
    if (threadIdx.x == 0) c.hit = 0xffffffffu;
    unsigned int pc;
    unsigned long long ps;
    block_excl_scan2(lc, ls, c, &pc, &ps);             // two barriers inside: hit init is visible
    unsigned int run_c = carry_cnt + pc;
    unsigned long long run_s = carry_sum + ps;
    int my_hit = -1;
    unsigned int hit_c = 0, bc = 0;
    unsigned long long hit_s = 0, bs = 0;
    if (mine) {
        for (int i = 0; i < nb && my_hit < 0; ++i) {
            const int b = n_bins - 1 - ((int)threadIdx.x * nb + i);
            const unsigned int cb = cnt[b];
            const unsigned long long sb = sums ? bin_sum64(*sums, b) : 0ull;
            const bool ok = cb > 0 && (by_sum ? (run_s + sb >= target)
                                              : ((unsigned long long)run_c + cb >= target));
            if (ok) { my_hit = b; hit_c = run_c; hit_s = run_s; bc = cb; bs = sb; }
            else { run_c += cb; run_s += sb; }
        }
    }
    // the first hit in descending bin order = the largest bin index that hit
    if (my_hit >= 0) atomicMin(&c.hit, 0xffffffffu - 1u - (unsigned int)my_hit);
    __syncthreads();
    if (my_hit >= 0 && c.hit == 0xffffffffu - 1u - (unsigned int)my_hit) {
        c.cnt_gt = hit_c;
        c.sum_gt = hit_s;
        c.bin_cnt = bc;
        c.bin_sum = bs;
        c.hit_bin = (unsigned int)my_hit;
    }
    __syncthreads();
}

constexpr int kCand = 128;   // this many tokens or fewer are resolved by direct comparison

// Last step of the descent when at most kCand tokens match the key prefix found so
// far: they are collected in shared memory and every candidate counts (and sums) the
// candidates above it.  A value is the threshold when the running total reaches the
// target once its copies are included, and no larger candidate value already does.
// On return: *key = the threshold's key; c.cnt_gt / c.sum_gt describe everything
// strictly above it, c.bin_cnt / c.bin_sum its copies.
__device__ void refine_direct(int L, const float *__restrict__ x, bool by_sum,
                              unsigned long long target, unsigned int prefix, unsigned int himask,
                              SelSmem &sm, SelCtl &c, unsigned int *key) {
    unsigned int *cand_key = sm.sum_lo, *fx_lo = sm.sum_hi, *fx_hi = sm.cnt_b;
    const unsigned int carry_c = c.cnt_gt;
    const unsigned long long carry_s = c.sum_gt;
    __syncthreads();                               // everyone holds the carries
    if (threadIdx.x == 0) c.n_cand = 0;            // slot counter while collecting
    __syncthreads();
    for (int jb = threadIdx.x; jb < L; jb += kSelThreads * kBatch) {
        float vals[kBatch];                        // the loads of a batch are in flight together
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int j = jb + u * kSelThreads;
            vals[u] = (j < L) ? x[j] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int j = jb + u * kSelThreads;
            const float v = vals[u];
            const unsigned int kx = float_key(v);
            if (j < L && (kx & himask) == prefix) {
                const unsigned int slot = atomicAdd(&c.n_cand, 1u);
                if (slot < (unsigned int)kCand) {
                    const unsigned long long fx = by_sum ? to_fx(v) : 0ull;
                    cand_key[slot] = kx;
                    fx_lo[slot] = (unsigned int)fx;
                    fx_hi[slot] = (unsigned int)(fx >> 32);
                }
            }
        }
    }
    __syncthreads();
    const unsigned int n = min(c.n_cand, (unsigned int)kCand);
    if (threadIdx.x < n) {
        const unsigned int mine = cand_key[threadIdx.x];
        unsigned int gt_c = 0, eq_c = 0;
        unsigned long long gt_s = 0;
        for (unsigned int i = 0; i < n; ++i) {
            const unsigned int kc = cand_key[i];                 // same address for the whole warp
            if (kc > mine) {
                ++gt_c;
                gt_s += ((unsigned long long)fx_hi[i] << 32) | fx_lo[i];
            }
            eq_c += (kc == mine);
        }
        const unsigned long long fx = ((unsigned long long)fx_hi[threadIdx.x] << 32) | fx_lo[threadIdx.x];
        const unsigned long long eq_s = fx * eq_c;
        bool hit;
        if (by_sum)
            hit = (carry_s + gt_s + eq_s >= target) && (gt_c == 0 || carry_s + gt_s < target);
        else
            hit = ((unsigned long long)carry_c + gt_c + eq_c >= target) &&
                  (gt_c == 0 || (unsigned long long)carry_c + gt_c < target);
        if (hit) {                                               // every copy writes the same values
            c.cnt_gt = carry_c + gt_c;
            c.sum_gt = carry_s + gt_s;
            c.bin_cnt = eq_c;
            c.bin_sum = eq_s;
            c.scan32[0] = mine;
        }
    }
    __syncthreads();
    *key = c.scan32[0];
    __syncthreads();
}

// One histogram level of the descent over the tokens whose key matches `prefix`
// under `himask`: `width` more bits at `shift`.  Updates prefix / himask and, in c,
// the carries (cnt_gt / sum_gt) and the chosen sub-bin's count / sum.
__device__ void refine_level(int L, const float *__restrict__ x, bool by_sum,
                             unsigned long long target, int shift, int width, unsigned int *prefix,
                             unsigned int *himask, SelSmem &sm, SelCtl &c) {
    const int n_bins = 1 << width;
    const unsigned int carry_c = c.cnt_gt;
    const unsigned long long carry_s = c.sum_gt;
    __syncthreads();
    for (int b = threadIdx.x; b < n_bins; b += kSelThreads) {
        sm.cnt_b[b] = 0; sm.sum_lo[b] = 0; sm.sum_hi[b] = 0;
    }
    __syncthreads();
    for (int jb = 0; jb < L; jb += kSelThreads * kBatch) {   // uniform trip count per warp
        float vals[kBatch];                        // the loads of a batch are in flight together
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int j = jb + u * kSelThreads + threadIdx.x;
            vals[u] = (j < L) ? x[j] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (jb + u * kSelThreads >= L) break;  // (the same for every thread)
            const int j = jb + u * kSelThreads + threadIdx.x;
            const float v = vals[u];
            const unsigned int kx = float_key(v);
            const bool act = j < L && (kx & *himask) == *prefix;
            hist_add(sm.cnt_b, by_sum ? &sm : nullptr, act, (kx >> shift) & (n_bins - 1),
                     (act && by_sum) ? to_fx(v) : 0ull);
        }
    }
    __syncthreads();
    find_bin(sm.cnt_b, by_sum ? &sm : nullptr, n_bins, by_sum, target, carry_c, carry_s, c);
    *prefix |= c.hit_bin << shift;                         // the prefix bin always contains a hit
    *himask |= (unsigned int)(n_bins - 1) << shift;
}

// The descent below the level-1 bin `b1` (which holds n_bin tokens): an 8-bit
// histogram level unless the bin is already small, then either direct comparison of
// the few tokens left or, if many tokens share 20 key bits (near-equal scores), a
// 12-bit histogram level over the rest of the key.
__device__ void refine(int L, const float *__restrict__ x, bool by_sum, unsigned long long target,
                       unsigned int b1, unsigned int n_bin, SelSmem &sm, SelCtl &c,
                       unsigned int *key) {
    unsigned int prefix = b1 << 20, himask = 0xfff00000u;
    if (n_bin > (unsigned int)kCand) {
        refine_level(L, x, by_sum, target, 12, 8, &prefix, &himask, sm, c);
        n_bin = c.bin_cnt;
    }
    if (n_bin <= (unsigned int)kCand) {
        refine_direct(L, x, by_sum, target, prefix, himask, sm, c, key);
    } else {
        refine_level(L, x, by_sum, target, 0, 12, &prefix, &himask, sm, c);
        *key = prefix;
    }
}

// Option outside the paper (the last positions join T whatever their score): how many
// of them the threshold leaves out, in front of this thread's chunk (.x) and in
// all (.y).  The same walk as the emission; kept out of line so that the
// ordinary call does not carry its instructions.
__device__ __noinline__ uint2 keep_last_extras(const float *__restrict__ rank, int j0, int j1, int f0,
                                               unsigned int thr_key, unsigned int eq_take, SelCtl &c) {
    unsigned int extra = 0, left = eq_take;
    for (int j = j0; j < j1; ++j) {
        const unsigned int key = float_key(rank[j]);
        bool keep = key > thr_key;
        if (!keep && key == thr_key && left > 0) { keep = true; --left; }
        extra += (!keep && j >= f0);
    }
    unsigned int extra_before;
    unsigned long long unused;
    block_excl_scan2(extra, 0ull, c, &extra_before, &unused);
    return make_uint2(extra_before, (unsigned int)block_sum64((unsigned long long)extra, c));
}

template <bool kKeepLast>   // (the option outside the paper is its own instantiation)
__global__ void __launch_bounds__(kSelThreads)
select_kernel(int L, const float *__restrict__ acc, const float *__restrict__ norm, float tau,
              uint32_t mode, int fixed_k, int32_t *__restrict__ k_out, int32_t *__restrict__ idx,
              float *__restrict__ kept_mass, GlobalHist *__restrict__ gh, int32_t *status_word) {
    extern __shared__ __align__(16) unsigned char sel_dyn[];
    SelSmem &sm = *reinterpret_cast<SelSmem *>(sel_dyn);
    __shared__ SelCtl c;

    // ---- every CTA: level-1 histogram of its 1024 tokens, then into the global one ----
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) {
        sm.cnt_b[b] = 0; sm.cnt_r[b] = 0; sm.sum_lo[b] = 0; sm.sum_hi[b] = 0;
    }
    if (threadIdx.x < 4) c.rng[threadIdx.x] = 0;
    grid_launch_dependents();
    grid_dependency_wait(acc, norm);   // the scores are the previous kernel's output
    const float *bud = (mode & ZIPVL_BUDGET_BY_NORM) ? norm : acc;
    const float *rank = (mode & ZIPVL_TOPK_BY_ACC) ? acc : norm;
    __syncthreads();
    // every CTA takes 1024 tokens; they meet in the global histogram
    bool bad_value = false;                        // a score that is negative or not a number
    const int row_end = min(L, (int)(blockIdx.x + 1) * kSelThreads);
    for (int jb = blockIdx.x * kSelThreads; jb < row_end; jb += kSelThreads * kBatch) {
        float vbs[kBatch], vrs[kBatch];            // the loads of a batch are in flight together
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int j = jb + u * kSelThreads + threadIdx.x;
            vbs[u] = (j < row_end) ? bud[j] : 0.f;
            vrs[u] = (j < row_end) ? rank[j] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (jb + u * kSelThreads >= row_end) break;   // (the same for every thread)
            const bool act = jb + u * kSelThreads + (int)threadIdx.x < row_end;
            const unsigned long long fxb = act ? to_fx(vbs[u]) : 0ull;
            bad_value |= act && (!(vbs[u] >= 0.f) || !(vrs[u] >= 0.f));
            hist_add(sm.cnt_b, &sm, act, float_key(vbs[u]) >> 20, fxb, &c.rng[0]);
            hist_add(sm.cnt_r, nullptr, act, float_key(vrs[u]) >> 20, 0ull, &c.rng[2]);
        }
    }
    // (such a score counts as zero in the sums and ranks by its bit pattern; the call
    // still completes, the caller is told)
    if (bad_value) report(status_word, ZIPVL_DEV_BAD_VALUE);
    __syncthreads();
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) {
        const unsigned int cb = sm.cnt_b[b], cr = sm.cnt_r[b];
        if (cb) {
            atomicAdd(&gh->cnt_b[b], cb);
            atomicAdd(&gh->sum_b[b], bin_sum64(sm, b));
        }
        if (cr) atomicAdd(&gh->cnt_r[b], cr);
    }
    if (threadIdx.x < 4) atomicMax(&gh->rng[threadIdx.x], c.rng[threadIdx.x]);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        c.is_last = (atomicAdd(&gh->ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!c.is_last) return;
    __threadfence();

    // ---- last CTA: the global histogram into shared memory ----
    for (int b = threadIdx.x; b < kBins; b += kSelThreads) {
        sm.cnt_b[b] = __ldcg(&gh->cnt_b[b]);
        sm.cnt_r[b] = __ldcg(&gh->cnt_r[b]);
        const unsigned long long s = __ldcg(&gh->sum_b[b]);
        sm.sum_lo[b] = (unsigned int)s;
        sm.sum_hi[b] = (unsigned int)(s >> 32);
    }
    if (threadIdx.x < 4) c.rng[threadIdx.x] = __ldcg(&gh->rng[threadIdx.x]);
    __syncthreads();

    // ---- the budget p (Eq. 7), then the threshold of the ranking score: the p-th
    // largest (Eq. 9).  Both are the same descent (by cumulative sum over the budget
    // score, by cumulative count over the ranking score), so they run as two passes of
    // one loop body: the second pass finds its instructions already fetched.
    const bool need_budget = !(fixed_k > 0) && (tau < 1.0f);
    unsigned int p = (fixed_k > 0) ? (unsigned int)min(fixed_k, L) : (unsigned int)L;
    unsigned int thr_key = 0, need_eq = L;
#pragma unroll 1
    for (int pass = need_budget ? 0 : 1; pass < 2; ++pass) {
        const bool by_sum = (pass == 0);
        if (!by_sum && p >= (unsigned int)L) break;
        const float *x = by_sum ? bud : rank;
        unsigned long long target = p;
        if (by_sum) {
            unsigned long long part = 0;
            for (int b = threadIdx.x; b < kBins; b += kSelThreads) part += bin_sum64(sm, b);
            const unsigned long long S_b = block_sum64(part, c);
            target = (unsigned long long)ceil((double)tau * (double)S_b);
        }
        const int r = by_sum ? 0 : 2;
        find_bin(by_sum ? sm.cnt_b : sm.cnt_r, by_sum ? &sm : nullptr, kBins, by_sum, target, 0u, 0ull, c,
                 (kBins - 1) - (int)c.rng[r + 1], (int)c.rng[r]);
        if (by_sum && c.hit == 0xffffffffu) {        // rounding let no prefix qualify: p stays L
            __syncthreads();
            continue;
        }
        unsigned int key;
        refine(L, x, by_sum, target, c.hit_bin, c.bin_cnt, sm, c, &key);
        if (by_sum) {
            // copies of the threshold value enter one at a time
            const unsigned long long v = c.bin_cnt ? c.bin_sum / c.bin_cnt : 0ull;
            unsigned long long need = 1;
            if (target > c.sum_gt && v > 0) need = (target - c.sum_gt + v - 1) / v;
            if (need < 1) need = 1;
            if (need > c.bin_cnt) need = c.bin_cnt;
            p = c.cnt_gt + (unsigned int)need;
            __syncthreads();
            // refine() reused cnt_b; the ranking counts of the next pass are untouched
        } else {
            thr_key = key;
            need_eq = p - c.cnt_gt;
        }
    }
    __syncthreads();

    // ---- emit T ascending: contiguous chunk of positions per thread ----
    const int per = (L + kSelThreads - 1) / kSelThreads;
    const int j0 = min(L, (int)threadIdx.x * per), j1 = min(L, j0 + per);
    unsigned int n_gt = 0, n_eq = 0;
    for (int jb = j0; jb < j1; jb += kBatch) {
        float vals[kBatch];                        // the loads of a batch are in flight together
#pragma unroll
        for (int u = 0; u < kBatch; ++u) vals[u] = (jb + u < j1) ? rank[jb + u] : 0.f;
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (jb + u < j1) {
                const unsigned int key = float_key(vals[u]);
                n_gt += key > thr_key;
                n_eq += key == thr_key;
            }
        }
    }
    // one scan of the pair (#equal, #greater) in front of this thread: of the copies of
    // the threshold the first need_eq (by position) are taken, so min(eq_before, need_eq)
    // of them precede this thread's chunk
    unsigned int eq_before;
    unsigned long long gt_before;
    block_excl_scan2(n_eq, (unsigned long long)n_gt, c, &eq_before, &gt_before);
    const bool all_sel = (p >= (unsigned int)L);
    const unsigned int eq_take = all_sel ? n_eq : min(n_eq, need_eq > eq_before ? need_eq - eq_before : 0u);
    unsigned int out = all_sel ? (unsigned int)j0 : (unsigned int)gt_before + min(eq_before, need_eq);
    unsigned int tot_sel = all_sel ? (unsigned int)L : p;
    // Option outside the paper: the last keep_last positions join T whatever their score.
    // Those of them that the threshold leaves out are counted per thread (the same walk
    // as the emission below) and scanned once more; without the option none of this runs.
    const unsigned int keep_last = mode >> 8;
    const int f0 = (kKeepLast && keep_last > 0 && !all_sel) ? max(0, L - (int)min(keep_last, (unsigned int)L)) : L;
    if (kKeepLast && f0 < L) {
        const uint2 ex = keep_last_extras(rank, j0, j1, f0, thr_key, eq_take, c);
        out += ex.x;
        tot_sel += ex.y;
    }
    unsigned int eq_left = eq_take;
    unsigned long long mass = 0, all = 0;
    for (int jb = j0; jb < j1; jb += kBatch) {
        float vr[kBatch], va[kBatch];              // the loads of a batch are in flight together
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            vr[u] = (jb + u < j1) ? rank[jb + u] : 0.f;
            va[u] = (jb + u < j1) ? acc[jb + u] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int j = jb + u;
            if (j >= j1) break;
            bool keep = true;
            if (p < (unsigned int)L) {
                const unsigned int key = float_key(vr[u]);
                keep = key > thr_key;
                if (!keep && key == thr_key && eq_left > 0) { keep = true; --eq_left; }
                if (kKeepLast) keep = keep || (j >= f0);
            }
            const unsigned long long fx = to_fx(va[u]);
            all += fx;
            if (keep) {
                idx[out++] = j;
                mass += fx;
            }
        }
    }
    for (int j = tot_sel + threadIdx.x; j < L; j += kSelThreads) idx[j] = -1;
    const unsigned long long kept = block_sum64(mass, c);
    const unsigned long long S_acc = block_sum64(all, c);
    if (threadIdx.x == 0) {
        *k_out = (int32_t)tot_sel;
        if (kept_mass) *kept_mass = S_acc ? (float)((double)kept / (double)S_acc) : 0.f;
    }
}


// ---------------------------------------------------------------------------------------
// Rows of up to 4096 tokens: one CTA of 256 threads with the whole row in registers.
//
// Thread t owns positions 16t .. 16t+15 (four 16-byte loads per score vector), so the row is
// read from memory once and the ascending emission is a walk over the thread's own registers.
// A block-wide step costs a barrier plus its warp shuffles once per warp, so the CTA is kept
// to eight warps and every phase to a few such steps; nothing loops over the row.
//
// The threshold searches are the ones described at the top of the file, with one change that
// matters at this size: the histogram levels adapt to the data.  Level 1 spreads its 4096
// bins over [smallest key, largest key] of the row instead of over the top 12 key bits (scores
// of one layer lie within a few octaves of each other, which is a few dozen of the fixed
// bins), so the crossing bin holds a handful of tokens instead of hundreds; each further
// level spreads 4096 bins over the crossing bin of the level before.  The descent ends when a
// bin holds one token or spans one key value (ties): two levels as a rule, three at most.
// ---------------------------------------------------------------------------------------
#ifndef ZIPVL_SOLO_THREADS
#define ZIPVL_SOLO_THREADS 512
#endif
constexpr int kSoloThreads = ZIPVL_SOLO_THREADS;
constexpr int kSoloPer = kSoloMax / kSoloThreads;   // 16 positions per thread
constexpr int kSoloWarps = kSoloThreads / 32;

struct SoloSmem {                      // dynamic shared memory
    // fixed-point sum of the budget score per bin as three words of 16-bit pieces (bits 0-15,
    // 16-31, 32 and up of each addend): three independent 32-bit adds without a carry to pass
    // on; exact while a bin's pieces stay below 2^32, i.e. for scores below 2^18
    unsigned int sum16[3][kBins];
    unsigned int cnt[kBins];
    unsigned int cnt_r[kBins];         // level 1 of the ranking score (filled in the same walk)
};
__device__ __forceinline__ void solo_add(SoloSmem &sm, unsigned int d, unsigned long long fx) {
    atomicAdd(&sm.cnt[d], 1u);
    atomicAdd(&sm.sum16[0][d], (unsigned int)fx & 0xffffu);
    atomicAdd(&sm.sum16[1][d], ((unsigned int)fx >> 16));
    atomicAdd(&sm.sum16[2][d], (unsigned int)(fx >> 32));
}
__device__ __forceinline__ unsigned long long solo_sum(const SoloSmem &sm, int b) {
    return (unsigned long long)sm.sum16[0][b] + ((unsigned long long)sm.sum16[1][b] << 16) +
           ((unsigned long long)sm.sum16[2][b] << 32);
}
struct SoloCtl {                       // static shared memory
    unsigned long long wsum[kSoloWarps], sum_gt, bin_sum;
    unsigned int wcnt[kSoloWarps], wmin[2][kSoloWarps], wmax[2][kSoloWarps];
    unsigned int hit, hit_bin, cnt_gt, bin_cnt, one_key;
    // the tokens of a sparsely filled crossing bin, resolved by one warp (see kDirect)
    unsigned int n_cand, cand_key[32];
    unsigned long long cand_fx[32];
};
constexpr unsigned int kDirect = 32;   // a crossing bin with this many tokens or fewer skips the next level

// block-wide (256 threads) exclusive prefix of a (count, sum) pair in thread order, and totals
__device__ __forceinline__ void solo_scan(unsigned int vc, unsigned long long vs, SoloCtl &c,
                                          unsigned int *pc, unsigned long long *ps,
                                          unsigned int *tc = nullptr, unsigned long long *ts = nullptr) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned int ic = vc;
    unsigned long long is = vs;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned int nc = __shfl_up_sync(0xffffffffu, ic, o);
        const unsigned long long ns = __shfl_up_sync(0xffffffffu, is, o);
        if (lane >= o) { ic += nc; is += ns; }
    }
    __syncthreads();                                   // earlier readers of wcnt / wsum are done
    if (lane == 31) { c.wcnt[w] = ic; c.wsum[w] = is; }
    __syncthreads();
    unsigned int bc = 0, allc = 0;
    unsigned long long bs = 0, alls = 0;
#pragma unroll
    for (int i = 0; i < kSoloWarps; ++i) {
        const unsigned int wc = c.wcnt[i];
        const unsigned long long wsm = c.wsum[i];
        if (i < w) { bc += wc; bs += wsm; }
        allc += wc; alls += wsm;
    }
    *pc = bc + ic - vc;
    *ps = bs + is - vs;
    if (tc) *tc = allc;
    if (ts) *ts = alls;
}

// One adaptive histogram level below the first: the range is the crossing bin of the level
// before, [base, base + 2^width_log2); a token whose key lies in it falls into bin
// (key - base) >> shift.
__device__ __forceinline__ bool solo_bin(unsigned int key, unsigned int base, int width_log2, int shift,
                                         unsigned int *d) {
    const unsigned int off = key - base;
    *d = off >> shift;
    return key >= base && (off >> width_log2) == 0u;
}

// The crossing bin from the top.  by_sum: first non-empty bin at which carry_sum + descending
// cumulative sum >= target; else the same by count.  Publishes hit (0xffffffff: none),
// hit_bin, cnt_gt / sum_gt (everything above the bin, carries included), bin_cnt / bin_sum.
// Three steps, each behind one barrier, so that only the warp that holds the crossing does
// the fine search: (1) every warp adds up its bins (kBins / warps, from the top), (2) warp 0
// walks the warp totals to the warp where the running total crosses, (3) that warp scans its
// lanes and the lane that crosses walks its own bins.
__device__ void solo_find_bin(const SoloSmem &sm, bool by_sum, unsigned long long target,
                              unsigned int carry_cnt, unsigned long long carry_sum, SoloCtl &c) {
    constexpr int kPer = kBins / kSoloThreads;         // bins per thread
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int b_top = kBins - 1 - (int)threadIdx.x * kPer;   // my bins: b_top, b_top-1, ...
    unsigned int cb[kPer];
    unsigned int lc = 0;
#pragma unroll
    for (int v4 = 0; v4 < kPer / 4; ++v4) {
        const uint4 q = *reinterpret_cast<const uint4 *>(&sm.cnt[b_top - 3 - 4 * v4]);
        cb[4 * v4 + 0] = q.w; cb[4 * v4 + 1] = q.z; cb[4 * v4 + 2] = q.y; cb[4 * v4 + 3] = q.x;
        lc += q.x + q.y + q.z + q.w;
    }
    unsigned long long ls = 0;
    if (by_sum && lc) {
#pragma unroll
        for (int i = 0; i < kPer; ++i)
            if (cb[i]) ls += solo_sum(sm, b_top - i);
    }
    // (1) warp totals: the count in one instruction, the sum as three 20-bit pieces
    const unsigned int wc = __reduce_add_sync(0xffffffffu, lc);
    unsigned long long wsum = 0;
    if (by_sum) {
        wsum = (unsigned long long)__reduce_add_sync(0xffffffffu, (unsigned int)ls & 0xfffffu) +
               ((unsigned long long)__reduce_add_sync(0xffffffffu, (unsigned int)(ls >> 20) & 0xfffffu) << 20) +
               ((unsigned long long)__reduce_add_sync(0xffffffffu, (unsigned int)(ls >> 40)) << 40);
    }
    __syncthreads();                                   // earlier readers of wcnt / wsum / hit are done
    if (lane == 0) { c.wcnt[w] = wc; c.wsum[w] = wsum; }
    __syncthreads();
    // (2) the warp in which the running total crosses
    if (threadIdx.x == 0) {
        unsigned int run_c = carry_cnt;
        unsigned long long run_s = carry_sum;
        unsigned int hit_w = 0xffffffffu;
        for (int i = 0; i < kSoloWarps; ++i) {
            const unsigned int tc = c.wcnt[i];
            const unsigned long long ts = c.wsum[i];
            const bool ok = tc > 0 && (by_sum ? (run_s + ts >= target) : ((unsigned long long)run_c + tc >= target));
            if (ok) { hit_w = i; break; }
            run_c += tc; run_s += ts;
        }
        c.hit = hit_w;                                 // (0xffffffff: no bin qualifies)
        c.cnt_gt = run_c;                              // everything above that warp's bins
        c.sum_gt = run_s;
    }
    __syncthreads();
    // (3) inside that warp
    if ((unsigned int)w == c.hit) {
        unsigned int ic = lc;
        unsigned long long is = ls;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int nc = __shfl_up_sync(0xffffffffu, ic, o);
            const unsigned long long ns = __shfl_up_sync(0xffffffffu, is, o);
            if (lane >= o) { ic += nc; is += ns; }
        }
        unsigned int run_c = c.cnt_gt + ic - lc;
        unsigned long long run_s = c.sum_gt + is - ls;
        const bool mine = lc > 0 && (by_sum ? (run_s + ls >= target) : ((unsigned long long)run_c + lc >= target));
        const unsigned int who = __ballot_sync(0xffffffffu, mine);
        if (who && lane == __ffs(who) - 1) {           // the first lane (highest bins) that crosses
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                if (cb[i]) {
                    const unsigned long long sb = by_sum ? solo_sum(sm, b_top - i) : 0ull;
                    const bool ok = by_sum ? (run_s + sb >= target) : ((unsigned long long)run_c + cb[i] >= target);
                    if (ok) {
                        c.cnt_gt = run_c;
                        c.sum_gt = run_s;
                        c.bin_cnt = cb[i];
                        c.bin_sum = sb;
                        c.hit_bin = (unsigned int)(b_top - i);
                        break;
                    }
                    run_c += cb[i]; run_s += sb;
                }
            }
        }
    }
    __syncthreads();
}

template <bool kKeepLast>
__global__ void __launch_bounds__(kSoloThreads)
select_solo_kernel(int L, const float *__restrict__ acc, const float *__restrict__ norm, float tau,
                   uint32_t mode, int fixed_k, int32_t *__restrict__ k_out, int32_t *__restrict__ idx,
                   float *__restrict__ kept_mass, int32_t *status_word) {
    extern __shared__ __align__(16) unsigned char sel_dyn[];
    SoloSmem &sm = *reinterpret_cast<SoloSmem *>(sel_dyn);
    __shared__ SoloCtl c;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    auto clear = [&](void *p, int bytes) {
        uint4 *z = reinterpret_cast<uint4 *>(p);
        for (int e = threadIdx.x; e < bytes / 16; e += kSoloThreads) z[e] = make_uint4(0, 0, 0, 0);
    };
    clear(&sm, sizeof(SoloSmem));      // while the previous kernel may still be running
    grid_launch_dependents();
    grid_dependency_wait(acc, norm);   // the scores are the previous kernel's output
    // one CTA per sequence of a batch: score rows, index lists and results are stacked
    acc += (size_t)blockIdx.x * L;
    norm += (size_t)blockIdx.x * L;
    idx += (size_t)blockIdx.x * L;
    k_out += blockIdx.x;
    if (kept_mass) kept_mass += blockIdx.x;
    const bool bud_is_norm = (mode & ZIPVL_BUDGET_BY_NORM) != 0, rank_is_acc = (mode & ZIPVL_TOPK_BY_ACC) != 0;
    // ---- the row into registers: positions j0 .. j0+15 (a vector that is not 16-byte aligned
    // is read element by element) ----
    const int j0 = (int)threadIdx.x * kSoloPer;
    float av[kSoloPer], nv[kSoloPer];
    const bool vec = (((uintptr_t)acc | (uintptr_t)norm) & 15u) == 0;
#pragma unroll
    for (int v4 = 0; v4 < kSoloPer / 4; ++v4) {
        const int j = j0 + 4 * v4;
        if (vec && j + 4 <= L) {
            const float4 a4 = *reinterpret_cast<const float4 *>(acc + j);
            const float4 n4 = *reinterpret_cast<const float4 *>(norm + j);
            av[4 * v4] = a4.x; av[4 * v4 + 1] = a4.y; av[4 * v4 + 2] = a4.z; av[4 * v4 + 3] = a4.w;
            nv[4 * v4] = n4.x; nv[4 * v4 + 1] = n4.y; nv[4 * v4 + 2] = n4.z; nv[4 * v4 + 3] = n4.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                av[4 * v4 + e] = (j + e < L) ? acc[j + e] : 0.f;
                nv[4 * v4 + e] = (j + e < L) ? norm[j + e] : 0.f;
            }
        }
    }
    // keys of the two scores, their ranges over the row, S of the budget score
    unsigned int kb[kSoloPer], kr[kSoloPer];
    unsigned int mn[2] = {0xffffffffu, 0xffffffffu}, mx[2] = {0u, 0u};
    unsigned long long my_sum = 0;
    bool bad_value = false;
#pragma unroll
    for (int e = 0; e < kSoloPer; ++e) {
        const float vb = bud_is_norm ? nv[e] : av[e], vr = rank_is_acc ? av[e] : nv[e];
        kb[e] = float_key(vb);
        kr[e] = float_key(vr);
        if (j0 + e < L) {
            mn[0] = min(mn[0], kb[e]); mx[0] = max(mx[0], kb[e]);
            mn[1] = min(mn[1], kr[e]); mx[1] = max(mx[1], kr[e]);
            my_sum += to_fx(vb);
            bad_value |= !(vb >= 0.f) || !(vr >= 0.f);
        }
    }
    if (bad_value) report(status_word, ZIPVL_DEV_BAD_VALUE);
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        mn[x] = __reduce_min_sync(0xffffffffu, mn[x]);
        mx[x] = __reduce_max_sync(0xffffffffu, mx[x]);
        if (lane == 0) { c.wmin[x][warp] = mn[x]; c.wmax[x][warp] = mx[x]; }
    }
    __syncthreads();                   // the ranges are in; the histograms are clear
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        mn[x] = 0xffffffffu; mx[x] = 0u;
#pragma unroll
        for (int i = 0; i < kSoloWarps; ++i) { mn[x] = min(mn[x], c.wmin[x][i]); mx[x] = max(mx[x], c.wmax[x][i]); }
    }
    auto first_shift = [](unsigned int lo, unsigned int hi) {
        const int bits = 32 - __clz(hi - lo);          // bits of the span (0 when all keys are equal)
        return bits > 12 ? bits - 12 : 0;
    };
    const bool need_budget = !(fixed_k > 0) && (tau < 1.0f);
    // ---- level 1 of both searches in one walk over the registers ----
    const int shift1[2] = {first_shift(mn[0], mx[0]), first_shift(mn[1], mx[1])};
#pragma unroll
    for (int e = 0; e < kSoloPer; ++e) {
        if (j0 + e < L) {
            if (need_budget) {
                solo_add(sm, (kb[e] - mn[0]) >> shift1[0], to_fx(bud_is_norm ? nv[e] : av[e]));
            }
            atomicAdd(&sm.cnt_r[(kr[e] - mn[1]) >> shift1[1]], 1u);
        }
    }
    unsigned int p = (fixed_k > 0) ? (unsigned int)min(fixed_k, L) : (unsigned int)L;
    unsigned int thr_key = 0, need_eq = L;
#pragma unroll 1
    for (int pass = need_budget ? 0 : 1; pass < 2; ++pass) {
        const bool by_sum = (pass == 0);
        if (!by_sum && p >= (unsigned int)L) break;
        const unsigned int *keys = by_sum ? kb : kr;
        unsigned long long target = p;
        if (by_sum) {
            unsigned int uc;
            unsigned long long us, S_b;
            solo_scan(0u, my_sum, c, &uc, &us, nullptr, &S_b);
            target = (unsigned long long)ceil((double)tau * (double)S_b);
        }
        unsigned int base = mn[pass], carry_c = 0;
        unsigned long long carry_s = 0;
        int shift = shift1[pass], width_log2 = 32;
        bool found = true;
        if (!by_sum) {
            // the ranking level 1 was counted into cnt_r: bring it to where the search reads
            __syncthreads();
            for (int e = threadIdx.x; e < kBins / 4; e += kSoloThreads)
                reinterpret_cast<uint4 *>(sm.cnt)[e] = reinterpret_cast<const uint4 *>(sm.cnt_r)[e];
        }
#pragma unroll 1
        for (int level = 0;; ++level) {
            if (level > 0) {
                // the next level: 4096 bins over the crossing bin of the one before
                __syncthreads();
                clear(sm.cnt, sizeof(sm.cnt));
                if (by_sum) clear(sm.sum16, sizeof(sm.sum16));
                __syncthreads();
#pragma unroll
                for (int e = 0; e < kSoloPer; ++e) {
                    unsigned int d;
                    if (j0 + e < L && solo_bin(keys[e], base, width_log2, shift, &d)) {
                        if (by_sum) solo_add(sm, d, to_fx(bud_is_norm ? nv[e] : av[e]));
                        else atomicAdd(&sm.cnt[d], 1u);
                    }
                }
            }
            __syncthreads();
            solo_find_bin(sm, by_sum, target, carry_c, carry_s, c);
            if (c.hit == 0xffffffffu) { found = false; break; }     // (rounding let no prefix qualify)
            if (shift == 0) { thr_key = base + c.hit_bin; break; }  // the bin is one key value
            if (c.bin_cnt <= kDirect) {
                // A handful of tokens in the crossing bin: their owners put them on a list and one
                // warp ranks them against each other -- lane i counts (and sums) the entries above
                // its own; the threshold is the largest key at which the running total, the copies
                // of that key included, reaches the target.  This replaces a whole histogram level.
                const unsigned int above_c = c.cnt_gt;
                const unsigned long long above_s = c.sum_gt;
                if (threadIdx.x == 0) c.n_cand = 0;
                __syncthreads();
#pragma unroll
                for (int e = 0; e < kSoloPer; ++e) {
                    unsigned int d;
                    const bool in = (level == 0) ? (d = (keys[e] - base) >> shift, true)
                                                 : solo_bin(keys[e], base, width_log2, shift, &d);
                    if (j0 + e < L && in && d == c.hit_bin) {
                        const unsigned int slot = atomicAdd(&c.n_cand, 1u);
                        if (slot < kDirect) {
                            c.cand_key[slot] = keys[e];
                            c.cand_fx[slot] = by_sum ? to_fx(bud_is_norm ? nv[e] : av[e]) : 0ull;
                        }
                    }
                }
                __syncthreads();
                if (threadIdx.x < 32) {
                    const unsigned int n = min(c.n_cand, kDirect);
                    const bool mine = (unsigned int)lane < n;
                    const unsigned int my_key = mine ? c.cand_key[lane] : 0u;
                    const unsigned long long my_fx = mine ? c.cand_fx[lane] : 0ull;
                    unsigned int gt_c = 0, eq_c = 0;
                    unsigned long long gt_s = 0;
                    for (unsigned int o = 0; o < n; ++o) {
                        const unsigned int ko = __shfl_sync(0xffffffffu, my_key, o);
                        const unsigned long long fo = __shfl_sync(0xffffffffu, my_fx, o);
                        if (ko > my_key) { ++gt_c; gt_s += fo; }
                        eq_c += (ko == my_key);
                    }
                    const unsigned long long eq_s = my_fx * eq_c;
                    bool hit;
                    if (by_sum) hit = (above_s + gt_s + eq_s >= target) && (gt_c == 0 || above_s + gt_s < target);
                    else hit = ((unsigned long long)above_c + gt_c + eq_c >= target) &&
                               (gt_c == 0 || (unsigned long long)above_c + gt_c < target);
                    if (mine && hit) {                          // (copies of one key write the same values)
                        c.cnt_gt = above_c + gt_c;
                        c.sum_gt = above_s + gt_s;
                        c.bin_cnt = eq_c;
                        c.bin_sum = eq_s;
                        c.one_key = my_key;
                    }
                }
                __syncthreads();
                thr_key = c.one_key;
                break;
            }
            base += c.hit_bin << shift;
            carry_c = c.cnt_gt;
            carry_s = c.sum_gt;
            width_log2 = shift;                        // (1..20: a bin of this level)
            shift = shift > 12 ? shift - 12 : 0;
        }
        if (by_sum) {
            if (found) {
                // copies of the threshold value enter one at a time
                const unsigned long long v = c.bin_cnt ? c.bin_sum / c.bin_cnt : 0ull;
                unsigned long long need = 1;
                if (target > c.sum_gt && v > 0) need = (target - c.sum_gt + v - 1) / v;
                if (need < 1) need = 1;
                if (need > c.bin_cnt) need = c.bin_cnt;
                p = c.cnt_gt + (unsigned int)need;
            }
            thr_key = 0;
        } else {
            need_eq = p - c.cnt_gt;
        }
    }
    __syncthreads();

    // ---- emit T ascending from the registers ----
    const bool all_sel = (p >= (unsigned int)L);
    unsigned int n_gt = 0, n_eq = 0;
#pragma unroll
    for (int e = 0; e < kSoloPer; ++e) {
        if (j0 + e < L) {
            n_gt += kr[e] > thr_key;
            n_eq += kr[e] == thr_key;
        }
    }
    unsigned int eq_before;
    unsigned long long gt_before;
    solo_scan(n_eq, (unsigned long long)n_gt, c, &eq_before, &gt_before);
    const unsigned int eq_take = all_sel ? n_eq : min(n_eq, need_eq > eq_before ? need_eq - eq_before : 0u);
    unsigned int out = all_sel ? (unsigned int)min(j0, L) : (unsigned int)gt_before + min(eq_before, need_eq);
    unsigned int tot_sel = all_sel ? (unsigned int)L : p;
    const unsigned int keep_last = mode >> 8;
    const int f0 = (kKeepLast && keep_last > 0 && !all_sel) ? max(0, L - (int)min(keep_last, (unsigned int)L)) : L;
    if (kKeepLast && f0 < L) {
        // the final positions the threshold leaves out, in front of this thread and in all
        unsigned int extra = 0, left = eq_take;
#pragma unroll
        for (int e = 0; e < kSoloPer; ++e) {
            if (j0 + e < L) {
                bool keep = kr[e] > thr_key;
                if (!keep && kr[e] == thr_key && left > 0) { keep = true; --left; }
                extra += (!keep && j0 + e >= f0);
            }
        }
        unsigned int extra_before, extra_all;
        unsigned long long unused;
        solo_scan(extra, 0ull, c, &extra_before, &unused, &extra_all);
        out += extra_before;
        tot_sel += extra_all;
    }
    unsigned int eq_left = eq_take;
    unsigned long long mass = 0, all = 0;
#pragma unroll
    for (int e = 0; e < kSoloPer; ++e) {
        const int j = j0 + e;
        if (j < L) {
            bool keep = true;
            if (!all_sel) {
                keep = kr[e] > thr_key;
                if (!keep && kr[e] == thr_key && eq_left > 0) { keep = true; --eq_left; }
                if (kKeepLast) keep = keep || (j >= f0);
            }
            const unsigned long long fx = to_fx(av[e]);
            all += fx;
            if (keep) {
                idx[out++] = j;
                mass += fx;
            }
        }
    }
    for (int j = tot_sel + threadIdx.x; j < L; j += kSoloThreads) idx[j] = -1;
    if (threadIdx.x == 0) *k_out = (int32_t)tot_sel;
    if (kept_mass) {
        unsigned int uc;
        unsigned long long us, kept, S_acc;
        solo_scan(0u, mass, c, &uc, &us, nullptr, &kept);
        solo_scan(0u, all, c, &uc, &us, nullptr, &S_acc);
        if (threadIdx.x == 0) *kept_mass = S_acc ? (float)((double)kept / (double)S_acc) : 0.f;
    }
}

}  // namespace

size_t select_ws_bytes() { return (sizeof(GlobalHist) + 255) & ~(size_t)255; }

zipvl_status launch_select(int L, const float *acc, const float *norm, float tau, uint32_t mode,
                           int fixed_k, int32_t *k_out, int32_t *idx, float *kept_mass, void *ws,
                           int32_t *status_word, cudaStream_t st, int n_seq) {
    if (L > kSoloMax && n_seq > 1) {
        // long rows: the multi-CTA kernel takes one sequence at a time (its workspace too)
        for (int z = 0; z < n_seq; ++z) {
            const zipvl_status sz = launch_select(L, acc + (size_t)z * L, norm + (size_t)z * L, tau, mode, fixed_k,
                                                  k_out + z, idx + (size_t)z * L, kept_mass ? kept_mass + z : nullptr,
                                                  ws, status_word, st, 1);
            if (sz != ZIPVL_OK) return sz;
        }
        return ZIPVL_OK;
    }
    if (L <= kSoloMax) {
        auto solo = (mode >> 8) ? select_solo_kernel<true> : select_solo_kernel<false>;
        cudaError_t es = cudaFuncSetAttribute(solo, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)sizeof(SoloSmem));
        if (es == cudaSuccess)
            es = launch_dependent(solo, dim3(n_seq), dim3(kSoloThreads), sizeof(SoloSmem), st, L, acc, norm, tau,
                                  mode, fixed_k, k_out, idx, kept_mass, status_word);
        if (es != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "select: launch: %s", cudaGetErrorString(es));
        count_launches(1);
        return check_launch("zipvl_select");
    }
    auto kernel = (mode >> 8) ? select_kernel<true> : select_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(SelSmem));
    const int grid = (L + kSelThreads - 1) / kSelThreads;
    if (e == cudaSuccess && grid > 1) e = cudaMemsetAsync(ws, 0, sizeof(GlobalHist), st);
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "select: %s", cudaGetErrorString(e));
    e = launch_dependent(kernel, dim3(grid), dim3(kSelThreads), sizeof(SelSmem), st, L, acc, norm, tau,
                         mode, fixed_k, k_out, idx, kept_mass, reinterpret_cast<GlobalHist *>(ws), status_word);
    if (e != cudaSuccess) return fail(ZIPVL_ERR_CUDA, "select: launch: %s", cudaGetErrorString(e));
    count_launches(1);
    return check_launch("zipvl_select");
}

}  // namespace zipvl
