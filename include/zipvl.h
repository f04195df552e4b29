/*
 * zipvl.h -- C ABI of the ZipVL per-layer hot path for NVIDIA B200 (sm_100a).
 *
 * ZipVL (arXiv 2410.08584) speeds up a vision-language model's attention by
 * (1) scoring every token with the attention of a few "probe" query rows,
 * (2) keeping, per layer, the smallest set of tokens whose accumulated score
 * reaches a fraction tau of the total, (3) running prefill attention over the
 * kept tokens only, (4) keeping only their keys / values in the cache and
 * (5) decoding against that compacted cache.  This library is those five
 * steps, each one call.
 *
 * Conventions shared by every call
 *   - Plain C.  No call throws, aborts or traps; each returns a zipvl_status.
 *     zipvl_last_error() gives the calling thread's last message.
 *   - OWNERSHIP: every tensor, index buffer, cache and workspace is DEVICE
 *     memory owned by the caller.  The library allocates no device memory and
 *     keeps no state between calls.  Only descriptor structs and scalars are
 *     HOST memory.  (The *_host convenience entry points at the end take host
 *     buffers and do allocate; they exist for end-to-end measurement.)
 *   - Every call is asynchronous on `stream` (a cudaStream_t passed as void*,
 *     NULL = the default stream) and never synchronises the host.
 *   - Layout: token-major, innermost dimension contiguous.  Q is
 *     [L, n_q_heads, head_dim]; K and V are [L, n_kv_heads, head_dim].  Query
 *     head h reads KV head h / (n_q_heads / n_kv_heads).  Token strides may be
 *     given in elements (0 = contiguous).  Base pointers are 16-byte aligned.
 *   - Problems seen on the device (an index out of range, a wait that ran out)
 *     are OR-ed into the caller's 4-byte device `status_word` (may be NULL) as
 *     ZIPVL_DEV_* bits; the offending access is skipped and the CUDA context
 *     stays usable.
 *   - Readings of the paper where it is silent are listed with each call.
 */
#ifndef ZIPVL_H_
#define ZIPVL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ZIPVL_OK = 0,
    ZIPVL_ERR_INVALID_ARG = 1, /* NULL pointer, bad size, tau outside (0,1], misalignment */
    ZIPVL_ERR_UNSUPPORTED = 2, /* head_dim / dtype / group size this build has no kernel for */
    ZIPVL_ERR_WORKSPACE = 3,   /* workspace smaller than zipvl_workspace_bytes() */
    ZIPVL_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (message has the text) */
    ZIPVL_ERR_TIMEOUT = 5,     /* reserved: host-visible form of ZIPVL_DEV_TIMEOUT */
    ZIPVL_ERR_BAD_INDEX = 6    /* reserved: host-visible form of ZIPVL_DEV_BAD_INDEX */
} zipvl_status;

/* bits OR-ed into the device status word */
#define ZIPVL_DEV_BAD_INDEX 1u /* an entry of idx / probe_pos / seq_lens was out of range */
#define ZIPVL_DEV_TIMEOUT 2u   /* a bounded wait inside a kernel ran out */
#define ZIPVL_DEV_CAPACITY 4u  /* k or a cache length exceeded the capacity given */
#define ZIPVL_DEV_BAD_VALUE 8u /* a score given to zipvl_select was negative or not a number */

#define ZIPVL_BF16 0
#define ZIPVL_F32 1
#define ZIPVL_F16 2 /* IEEE half: same kernels as bf16, fp32 accumulation */

/* operations, for zipvl_workspace_bytes() */
#define ZIPVL_OP_SCORE 0
#define ZIPVL_OP_SELECT 1
#define ZIPVL_OP_SPARSE_PREFILL 2
#define ZIPVL_OP_COMPACT_KV 3
#define ZIPVL_OP_DECODE 4

/* One attention layer of one sequence (HOST struct). */
typedef struct {
    int32_t L;             /* tokens n */
    int32_t n_q_heads;     /* Hq */
    int32_t n_kv_heads;    /* Hkv, divides Hq */
    int32_t head_dim;      /* 64, 96 or 128: all three run on the tensor cores in 16-bit storage */
    int32_t dtype;         /* ZIPVL_BF16 / ZIPVL_F16 (tensor-core path) or ZIPVL_F32 (true fp32 path) */
    int32_t reserved;
    int64_t q_stride_tok;  /* elements between tokens of Q; 0 = n_q_heads*head_dim */
    int64_t kv_stride_tok; /* elements between tokens of K and V; 0 = n_kv_heads*head_dim */
    float softmax_scale;   /* 0 = 1/sqrt(head_dim) */
    int32_t reserved2;
} zipvl_layer;

/* Ragged decode batch (HOST struct). */
typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim, dtype;
    float softmax_scale; /* 0 = 1/sqrt(head_dim) */
} zipvl_decode_desc;

const char *zipvl_status_string(zipvl_status s);
const char *zipvl_last_error(void); /* thread-local text of the last failure */
int32_t zipvl_version(void);
/* Number of CUDA kernels this library has launched in this process so far. */
uint64_t zipvl_launch_count(void);

/* Bytes of device workspace `op` needs for this layer.  `n_probe` matters to
 * SCORE only; for DECODE pass the batch size in `batch` and the largest cache
 * length any request can reach in layer->L.  Returns 0 on a bad argument. */
size_t zipvl_workspace_bytes(int32_t op, const zipvl_layer *layer, int32_t n_probe, int32_t batch);

/*
 * zipvl_score -- probe attention, accumulated and normalised token scores.
 * Paper: supplementary Eq. A (probe attention), Eq. 6 (accumulated score =
 * column sum), Eq. 8 (normalised score = column sum / nnz).
 *
 *   For every query head h and probe row r at position c = probe_pos[r]:
 *     A[h,r,j] = softmax over j <= c of scale * <Q[c,h,:], K[j,g,:]>, 0 for j > c
 *   acc[j]  = sum_h sum_r A[h,r,j]
 *   norm[j] = acc[j] / (n_q_heads * nnz[j]),  nnz[j] = #{ r : probe_pos[r] >= j }
 *   *total  = sum_j acc[j]   (equals n_probe * n_q_heads up to rounding)
 *
 * Readings: the probe rows carry the causal mask of Eq. 2 (only the mask
 * creates the zeros Eq. 8's nnz counts); nnz is structural; scores of all heads
 * are summed so that a layer has one token set; scale is 1/sqrt(head_dim).
 * A column no probe can see gets acc = norm = 0.
 *
 * q, k: device tensors (layout above).  probe_pos: device int32[n_probe],
 * strictly ascending; which rows to probe (the paper uses 64 recent + 64
 * random) is the caller's choice.  Entries outside [0,L) are skipped and
 * reported as ZIPVL_DEV_BAD_INDEX.  acc, norm: device float[L], written.
 * total: device double[1] or NULL.  ws: zipvl_workspace_bytes(ZIPVL_OP_SCORE).
 * The attention matrix A never reaches global memory.  Two calls on the same inputs give the
 * same bits (no floating-point sum depends on the order in which thread blocks finish).
 */
zipvl_status zipvl_score(const zipvl_layer *layer, const void *q, const void *k,
                         const int32_t *probe_pos, int32_t n_probe, float *acc, float *norm,
                         double *total, void *ws, size_t ws_bytes, int32_t *status_word,
                         void *stream);

/* mode bits for zipvl_select: which score fixes the budget p (Eq. 7) and which
 * picks the set T (Eq. 9).  0 = the paper's pairing: accumulated -> p,
 * normalised -> T.  The other pairings are the paper's Table B ablation. */
#define ZIPVL_BUDGET_BY_NORM 1u
#define ZIPVL_TOPK_BY_ACC 2u
/* An option outside the paper, which does not say whether the final positions
 * (whose outputs produce the first generated token) must survive: with
 * mode | ZIPVL_KEEP_LAST(r) the set written is the union of Eq. 9's T and the
 * last r positions, and *k_out is the size of that union (at most p + r). */
#define ZIPVL_KEEP_LAST(r) ((uint32_t)(r) << 8)
#define ZIPVL_KEEP_LAST_MAX 0xFFFFFFu

/*
 * zipvl_select -- layer-adaptive budget and important-token set.
 * Paper: Eq. 7 (p = fewest top-scored tokens whose score sum reaches tau x
 * total), Eq. 9 (T = top-p indices of the normalised score).
 *
 *   S = sum_j acc[j];  sort acc descending;  C_i = sum of the first i;
 *   p = min{ i >= 1 : C_i >= tau * S };  tau >= 1 gives p = L.
 *   T = the p positions with the largest norm[j], ties toward the smaller
 *       position, written to idx in ASCENDING position (causal order);
 *   idx[p..L) = -1.  *k_out = p.  *kept_mass = sum_{j in T} acc[j] / S.
 *
 * Readings: Eq. 7's target "tau x n" is tau x S (the paper's own remark is
 * that the scores sum to n); fixed_k > 0 replaces the adaptive p (fixed-ratio
 * ablation, Table 3) and is clamped to L.  Sums are taken in 2^-34 fixed point,
 * so results do not depend on thread order and repeat bit for bit.  The call
 * enqueues one kernel, preceded for rows longer than 4096 tokens by one memset
 * of its workspace.  mode: ZIPVL_BUDGET_BY_NORM, ZIPVL_TOPK_BY_ACC, ZIPVL_KEEP_LAST(r) or'ed
 * together; any other bit is ZIPVL_ERR_INVALID_ARG.
 *
 * acc, norm: device float[L], non-negative; a negative or NaN entry counts as zero in
 * the sums, ranks by its bit pattern and is reported as ZIPVL_DEV_BAD_VALUE.  Sums are
 * exact for scores below 2^18 (a column sum of attention is at most n_probe x n_q_heads).
 * k_out: device int32[1].
 * idx: device int32[L].  kept_mass: device float[1] or NULL.
 * ws: zipvl_workspace_bytes(ZIPVL_OP_SELECT).  L <= 2^20.
 */
zipvl_status zipvl_select(int32_t L, const float *acc, const float *norm, float tau,
                          uint32_t mode, int32_t fixed_k, int32_t *k_out, int32_t *idx,
                          float *kept_mass, void *ws, size_t ws_bytes, int32_t *status_word,
                          void *stream);

#define ZIPVL_OUT_PADDED 0  /* out is [L, Hq, d]; rows outside T are zero-filled by the call */
#define ZIPVL_OUT_COMPACT 1 /* out is [k, Hq, d], row i belongs to token idx[i] */

/*
 * zipvl_sparse_prefill -- causal attention over the important tokens only.
 * Paper: Algorithm 1, "O = FlashAttention(Q[T], K[T], V[T])"; Eq. 2 on the
 * gathered tokens; Sec. 3.2: outputs of the other tokens are padded.
 *
 *   for i in [0,k), head h:  w_j = softmax over j <= i of
 *       scale * <Q[T_i,h,:], K[T_j,g,:]>;   o = sum_j w_j V[T_j,g,:]
 *   PADDED: out[T_i,h,:] = o and every row outside T = 0.  COMPACT: out[i,h,:] = o.
 *
 * Reading: padding is zeros.  idx: device int32, ascending (as zipvl_select
 * writes it); k_dev: device int32[1], read on the device, so no host sync sits
 * between select and prefill; k_max: host upper bound on k used to size the
 * launch (pass L if unknown).  k > k_max is clamped and reported as
 * ZIPVL_DEV_CAPACITY.  out has the layer's dtype, contiguous.
 * An entry of idx[0..k) outside [0, L) is reported as ZIPVL_DEV_BAD_INDEX: no memory
 * is read or written for it (its output row is left alone, the rows of dropped
 * tokens next to it are not cleared) and it stands in the attention of the later
 * rows as an all-zero key and value.  k = 0 writes an all-zero PADDED output.
 */
zipvl_status zipvl_sparse_prefill(const zipvl_layer *layer, const void *q, const void *k,
                                  const void *v, const int32_t *idx, const int32_t *k_dev,
                                  int32_t k_max, void *out, int32_t out_mode, void *ws,
                                  size_t ws_bytes, int32_t *status_word, void *stream);

/*
 * zipvl_compact_kv -- keep only the important tokens' keys and values.
 * Paper: Algorithm 1, "K = K[T], V = V[T]" (Sec. 3.2, KV cache eviction).
 *
 *   k_cache[i,:,:] = k[T_i,:,:], v_cache likewise, bit for bit, i in [0,k);
 *   *len_out = k.   Caches are contiguous [capacity, Hkv, d].
 * k > min(k_max, capacity) is clamped and reported as ZIPVL_DEV_CAPACITY.
 */
zipvl_status zipvl_compact_kv(const zipvl_layer *layer, const void *k, const void *v,
                              const int32_t *idx, const int32_t *k_dev, int32_t k_max,
                              void *k_cache, void *v_cache, int32_t capacity, int32_t *len_out,
                              int32_t *status_word, void *stream);

/*
 * zipvl_sparse_prefill_compact -- zipvl_sparse_prefill and zipvl_compact_kv in one call.
 * Paper: Algorithm 1 does both for every layer, one after the other
 * ("O = FlashAttention(Q[T], K[T], V[T])", then "K = K[T], V = V[T]"); both depend only
 * on T.  Results are those of the two calls: out as zipvl_sparse_prefill writes it,
 * k_cache / v_cache / *len_out as zipvl_compact_kv writes them, bit for bit.
 * For 16-bit storage (head_dim 64, 96 or 128) and a token stride that is a multiple of 16 bytes the copy
 * runs inside the attention kernel (spare warps of each attention CTA copy the key
 * and value rows of that CTA's kept tokens), which takes the compaction off the
 * layer's critical path; other shapes run the two kernels back to back.
 * Arguments as in the two calls; ws: zipvl_workspace_bytes(ZIPVL_OP_SPARSE_PREFILL).
 * k > k_max is clamped for the attention, k > capacity for the caches; both are
 * reported as ZIPVL_DEV_CAPACITY.  One difference in an error case: a cache row
 * whose index is out of range (reported as ZIPVL_DEV_BAD_INDEX) is written as
 * zeros by the in-kernel copy, where zipvl_compact_kv leaves it untouched.
 */
zipvl_status zipvl_sparse_prefill_compact(const zipvl_layer *layer, const void *q, const void *k,
                                          const void *v, const int32_t *idx, const int32_t *k_dev,
                                          int32_t k_max, void *out, int32_t out_mode, void *k_cache,
                                          void *v_cache, int32_t capacity, int32_t *len_out, void *ws,
                                          size_t ws_bytes, int32_t *status_word, void *stream);

/*
 * Several sequences per call.  (The paper treats one sequence; Algorithm 1 is run for every
 * layer of every sequence, and sequences are independent, so a batch is the same arithmetic
 * per sequence.)  A batch is n_seq sequences of ONE shape (the zipvl_layer), stacked:
 * sequence z of Q starts q_stride_seq elements after sequence z-1 (0 = L x token stride,
 * i.e. [n_seq, L, Hq, d] without gaps), K and V likewise with kv_stride_seq.  Everything
 * per-sequence is stacked without gaps: probe_pos [n_seq, n_probe], acc / norm / idx
 * [n_seq, L], k_out / k_dev / len_out / total / kept_mass [n_seq], out [n_seq, L or k_max,
 * Hq, d], caches [n_seq, capacity, Hkv, d].  Results per sequence are those of the
 * single-sequence calls, bit for bit.  Where the tensor-core kernels apply, a batch is one
 * launch whose grid spans the sequences (short sequences alone cannot fill the GPU);
 * other shapes run sequence by sequence inside the call.
 */
typedef struct {
    int32_t n_seq;
    int32_t reserved;
    int64_t q_stride_seq;  /* elements between sequences of Q; 0 = L * token stride */
    int64_t kv_stride_seq; /* elements between sequences of K and of V; 0 = L * token stride */
} zipvl_batch;

/* zipvl_workspace_bytes for the batched calls (only ZIPVL_OP_SCORE grows with n_seq). */
size_t zipvl_workspace_bytes_batch(int32_t op, const zipvl_layer *layer, int32_t n_probe, int32_t n_seq);

/* zipvl_score for a batch (Eq. A, Eq. 6, Eq. 8 per sequence). */
zipvl_status zipvl_score_batch(const zipvl_layer *layer, const zipvl_batch *batch, const void *q,
                               const void *k, const int32_t *probe_pos, int32_t n_probe, float *acc,
                               float *norm, double *total, void *ws, size_t ws_bytes,
                               int32_t *status_word, void *stream);

/* zipvl_select for a batch of n_seq score rows of length L (Eq. 7, Eq. 9 per sequence; one
 * tau, mode and fixed_k for all). */
zipvl_status zipvl_select_batch(int32_t L, int32_t n_seq, const float *acc, const float *norm, float tau,
                                uint32_t mode, int32_t fixed_k, int32_t *k_out, int32_t *idx,
                                float *kept_mass, void *ws, size_t ws_bytes, int32_t *status_word,
                                void *stream);

/* zipvl_sparse_prefill for a batch (Algorithm 1's attention per sequence); with k_cache !=
 * NULL also zipvl_compact_kv, as zipvl_sparse_prefill_compact does (then v_cache and len_out
 * are required and capacity >= 1). */
zipvl_status zipvl_sparse_prefill_batch(const zipvl_layer *layer, const zipvl_batch *batch, const void *q,
                                        const void *k, const void *v, const int32_t *idx,
                                        const int32_t *k_dev, int32_t k_max, void *out, int32_t out_mode,
                                        void *k_cache, void *v_cache, int32_t capacity, int32_t *len_out,
                                        void *ws, size_t ws_bytes, int32_t *status_word, void *stream);

/*
 * zipvl_decode -- one decoding step over the kept cache, ragged batch.
 * Paper: Algorithm 2; Eq. 4 (append the new key / value), Eq. 5 (attention of
 * the single query over the whole cache).  Nothing is evicted while decoding.
 *
 *   request b: cache rows live at k_cache + cache_off[b] (elements), row pitch
 *   Hkv*d, at most capacity[b] rows, seq_lens[b] of them valid.
 *   If k_new != NULL: row seq_lens[b] <- k_new[b], v_new[b]; seq_lens[b] += 1.
 *   out[b,h,:] = sum_j softmax_j(scale * <q[b,h,:], Kc_b[j,g,:]>) * Vc_b[j,g,:]
 *   over all seq_lens[b] rows (after the append), no mask.
 *
 * q, out: device [B, Hq, d]; k_new, v_new: device [B, Hkv, d] or both NULL;
 * cache_off: device int64[B] (multiples of 8 elements); capacity, seq_lens:
 * device int32[B].  max_len: host upper bound on any seq_lens[b] after the
 * append; sizes the launch and the workspace.  A request whose cache is full
 * is not appended to and reports ZIPVL_DEV_CAPACITY; a request with zero rows
 * writes zeros.  A request with seq_lens[b] < 0 or > capacity[b], or whose
 * cache_off[b] is not a multiple of 16 bytes, is skipped as a whole (nothing of
 * its cache is read or written, its output is zeros, its length stays) and
 * reported as ZIPVL_DEV_BAD_INDEX.  The call enqueues two kernels (the second merges the cache chunks).
 * Query heads per kv head (Hq / Hkv): up to 8 for any dtype; up to 32 in 16-bit storage,
 * where grouped heads run on the tensor cores (the query heads of a kv
 * head are the rows of an MMA tile, so grouped-query attention stays bound by HBM instead of by
 * multiply-adds): one CTA per chunk of a request's cache for small problems, a persistent launch
 * (one CTA per SM over an equal share of all key/value tiles) for large ones.  Same results
 * contract on every path; ZIPVL_DECODE_KERNEL=simt|tc|tcp in the environment forces the
 * CUDA-core, the chunked or the persistent tensor-core kernel where it applies.
 */
zipvl_status zipvl_decode(const zipvl_decode_desc *desc, const void *q, const void *k_new,
                          const void *v_new, void *k_cache, void *v_cache,
                          const int64_t *cache_off, const int32_t *capacity, int32_t *seq_lens,
                          int32_t max_len, void *out, void *ws, size_t ws_bytes,
                          int32_t *status_word, void *stream);

/*
 * zipvl_decode_paged -- zipvl_decode over a paged cache.
 * Paper: Algorithm 2, Eq. 4-5, as zipvl_decode; only the storage of the kept cache differs
 * (serving systems keep caches that grow token by token in fixed-size pages of a shared pool).
 *
 *   k_pages, v_pages: device pools [n_pages, page_rows, Hkv, d]; page_rows a power of two
 *   from 16 to 1024.  block_table: device int32 [batch, table_stride]; request b's row r is
 *   row r % page_rows of page block_table[b * table_stride + r / page_rows].
 *   capacity[b]: rows request b may hold (its pages x page_rows); table_stride must cover
 *   max_len rows.  Everything else as zipvl_decode (append at row seq_lens[b], attention over
 *   all rows, ZIPVL_DEV_CAPACITY for a full cache).  A page number outside [0, n_pages) is
 *   reported as ZIPVL_DEV_BAD_INDEX and its rows are left out of the attention.
 * ws: zipvl_workspace_bytes(ZIPVL_OP_DECODE) as for zipvl_decode.
 */
zipvl_status zipvl_decode_paged(const zipvl_decode_desc *desc, const void *q, const void *k_new,
                                const void *v_new, void *k_pages, void *v_pages,
                                const int32_t *block_table, int32_t table_stride,
                                int32_t page_rows, int32_t n_pages, const int32_t *capacity,
                                int32_t *seq_lens, int32_t max_len, void *out, void *ws,
                                size_t ws_bytes, int32_t *status_word, void *stream);

/*
 * zipvl_quantize_kv, zipvl_decode_quant -- the mixed-precision KV cache.
 * Paper: Sec. 4.3 / Table 3 (the adaptive token set drives a mixed-precision cache: "important
 * tokens are quantized to 4-bit, while other tokens are quantized to 2-bit"); decode as
 * Algorithm 2, Eq. 4-5.  The paper takes the quantiser from the work it cites; the reading
 * built here: no token is evicted; keys and values are quantised per (token, KV head) over the
 * head_dim channels, scale = (max - min) / (2^b - 1), code = clip(rint((x - min) * (1 / scale)),
 * 0, 2^b - 1), with scale and min rounded to the storage type and kept beside the codes (each step
 * a correctly rounded fp32 operation).  The cache of a sequence is two blocks -- softmax
 * attention does not depend on the order of the cached rows:
 *   "hi": the tokens of T in T's order at 4 bits; k_hi, v_hi: [cap_hi, Hkv, d/2] bytes,
 *         params_hi: [cap_hi, Hkv, 4] storage-type values (k scale, k min, v scale, v min);
 *   "lo": the other tokens, ascending, at 2 bits; k_lo, v_lo: [cap_lo, Hkv, d/4] bytes, params_lo alike.
 *   Channel c of a row sits in byte c*b/8 at bit (c*b)%8.  lens: device int32[2] = rows in hi, lo.
 * zipvl_quantize_kv builds the blocks from K, V and the token set (idx ascending, k_dev on the
 * device, k_max the host's bound) and writes lens_out; a block that is too small is filled to
 * its capacity and ZIPVL_DEV_CAPACITY reported.  zipvl_decode_quant is one decode step of ONE
 * request (desc->batch == 1): if k_new != NULL the new key / value ([Hkv,d]) are quantised at
 * 4 bits and appended to the hi block (lens[0] += 1; a full block: ZIPVL_DEV_CAPACITY, no
 * append); out[h,:] = softmax attention of q[h,:] over all dequantised rows.  max_len: host
 * bound on lens[0] + lens[1] after the append; ws: zipvl_workspace_bytes(ZIPVL_OP_DECODE) for
 * batch 1 and L = max_len.  16-bit storage types, head_dim 64 or 128, 1, 2 or 4 query heads per
 * KV head, at most 64 KV heads.  The call enqueues two kernels (three with an append).
 */
zipvl_status zipvl_quantize_kv(const zipvl_layer *layer, const void *k, const void *v, const int32_t *idx,
                               const int32_t *k_dev, int32_t k_max, void *k_hi, void *v_hi,
                               void *params_hi, int32_t cap_hi, void *k_lo, void *v_lo, void *params_lo,
                               int32_t cap_lo, int32_t *lens_out, int32_t *status_word, void *stream);
zipvl_status zipvl_decode_quant(const zipvl_decode_desc *desc, const void *q, const void *k_new,
                                const void *v_new, void *k_hi, void *v_hi, void *params_hi, int32_t cap_hi,
                                void *k_lo, void *v_lo, void *params_lo, int32_t cap_lo, int32_t *lens,
                                int32_t max_len, void *out, void *ws, size_t ws_bytes,
                                int32_t *status_word, void *stream);

/*
 * zipvl_decode_quant_batch -- zipvl_decode_quant for desc->batch requests in one call.
 * (Algorithm 2, Eq. 4-5 per request; the requests are independent.)
 * caches: DEVICE array of desc->batch entries, one request's blocks each (all pointers DEVICE,
 * laid out and aligned as zipvl_decode_quant takes them; lens: that request's int32[2]).
 * q, out: [batch, Hq, d]; k_new, v_new: [batch, Hkv, d] or both NULL; max_len: host bound on
 * any request's lens[0] + lens[1] after the append; ws: zipvl_workspace_bytes(ZIPVL_OP_DECODE)
 * for this batch and L = max_len.  The table lives on the device, so its entries are checked
 * there: a request whose entry has a NULL or misaligned block, or a capacity below 1, is
 * skipped (nothing appended, an output of zeros) and reported as ZIPVL_DEV_BAD_INDEX; a full
 * 4-bit block as ZIPVL_DEV_CAPACITY, per request.  Same shapes as zipvl_decode_quant.
 * The call enqueues two kernels (three with an append), whatever the batch.
 */
typedef struct zipvl_quant_cache {
    void *k_hi, *v_hi, *params_hi;   /* the 4-bit block */
    void *k_lo, *v_lo, *params_lo;   /* the 2-bit block */
    int32_t *lens;                   /* rows in hi, lo */
    int32_t cap_hi, cap_lo;
} zipvl_quant_cache;

zipvl_status zipvl_decode_quant_batch(const zipvl_decode_desc *desc, const void *q, const void *k_new,
                                      const void *v_new, const zipvl_quant_cache *caches, int32_t max_len,
                                      void *out, void *ws, size_t ws_bytes, int32_t *status_word,
                                      void *stream);

/*
 * zipvl_decode_noalloc -- zipvl_decode for callers that cannot allocate.
 * (The paper has no counterpart: this is a deployment variant of the decode
 * step, same arithmetic, same kernels.)
 *
 * Some callers have no way to hand the library a workspace: code running
 * under a memory manager that forbids cudaMalloc after start-up, a plugin whose
 * host gives it only input and output buffers, a serving loop whose memory pool
 * is already carved up.  For them the split-KV partial results live in an
 * 8 MiB array that is part of the library image on the device (every GPU that
 * loads the library holds it until the process exits).  The call allocates
 * nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *
 * Same arguments and results as zipvl_decode, minus ws / ws_bytes.  Limit:
 * batch * n_q_heads * ceil(max_len / chunk) * (head_dim + 2) * 4 bytes must fit
 * in 8 MiB, where chunk is the number of cache rows the library gives one thread
 * block (a power of two from 32 to 512, growing with the problem) -- e.g. batch
 * 16, 32 heads, head_dim 128 fits up to max_len 15872.  A shape the grouped-query
 * tensor-core kernels take (16-bit storage, 2 to 32 query heads per kv head) needs 4 * (ceil(max_len / chunk) + 1) such slots per query head plus
 * 4 bytes per (request, query head).  Larger problems are refused with
 * ZIPVL_ERR_WORKSPACE and a message; use zipvl_decode with a workspace.
 *
 * The first call on each device looks up the array's device address (with that
 * device current) and caches it for the life of the process; make that first
 * call before starting any stream capture.  The cached address belongs to the
 * device's primary context: after cudaDeviceReset it is stale and this entry
 * point must not be used again in the process.  All calls share the one array and it keeps the previous
 * call's contents: nothing in it has to start at zero, every slot a call reads
 * was written by that same call.  Two calls that overlap on the GPU
 * (different streams, no ordering between them) race on it: order them.
 */
zipvl_status zipvl_decode_noalloc(const zipvl_decode_desc *desc, const void *q,
                                  const void *k_new, const void *v_new, void *k_cache,
                                  void *v_cache, const int64_t *cache_off,
                                  const int32_t *capacity, int32_t *seq_lens, int32_t max_len,
                                  void *out, int32_t *status_word, void *stream);

/*
 * zipvl_prefill_layer_host -- Algorithm 1 end to end from HOST buffers.
 * Copies q, k, v and probe_pos to the device, runs score -> select ->
 * sparse_prefill (PADDED) -> compact_kv, and copies k, idx, the padded output
 * and the compacted caches back.  Allocates and frees its own device memory
 * and synchronises; it exists so that a caller with host data (and the
 * end-to-end benchmark) can use the path with one call.  All pointers HOST.
 * out: [L,Hq,d]; k_cache_out / v_cache_out: [L,Hkv,d] capacity, first *k_out
 * rows valid; idx_out: int32[L].  Any output pointer may be NULL to skip it.
 */
zipvl_status zipvl_prefill_layer_host(const zipvl_layer *layer, const void *q, const void *k,
                                      const void *v, const int32_t *probe_pos, int32_t n_probe,
                                      float tau, int32_t *k_out, int32_t *idx_out, void *out,
                                      void *k_cache_out, void *v_cache_out);

/*
 * zipvl_layer_step_host -- zipvl_prefill_layer_host followed by one decode step, from HOST
 * buffers: Algorithm 1 for the layer, then Algorithm 2 for one new token on the cache the
 * call has just compacted (the new key / value are appended behind the kept rows, Eq. 4,
 * and the new query attends over all of them, Eq. 5).  q_new: [Hq,d]; k_new, v_new:
 * [Hkv,d]; decode_out: [Hq,d]; all HOST, all four given or all four NULL (then this is
 * zipvl_prefill_layer_host).  The caches copied back hold the kept rows, not the appended
 * one.  At most 8 query heads per KV head, as for zipvl_decode.
 */
zipvl_status zipvl_layer_step_host(const zipvl_layer *layer, const void *q, const void *k,
                                   const void *v, const int32_t *probe_pos, int32_t n_probe,
                                   float tau, int32_t *k_out, int32_t *idx_out, void *out,
                                   void *k_cache_out, void *v_cache_out, const void *q_new,
                                   const void *k_new, const void *v_new, void *decode_out);

/*
 * zipvl_release_host_scratch -- give back the device memory zipvl_prefill_layer_host
 * keeps between calls.  (No counterpart in the paper.)  That call takes its device
 * scratch from a memory pool of the library's own, one per device, which keeps freed
 * memory for the next call instead of returning it to the driver; this function trims
 * the current device's pool to zero.  Safe to call at any time; a no-op if
 * zipvl_prefill_layer_host never ran on the device.
 */
zipvl_status zipvl_release_host_scratch(void);

/*
 * zipvl_selftest_wait_timeout -- run a bounded device wait out, on purpose and harmlessly.
 * (No counterpart in the paper: a check of the library's own failure handling.)
 * Every wait inside the tensor-core kernels gives up after a fixed number of polls, raises
 * its thread block's abort flag, lets all warps leave through the common exit and reports
 * ZIPVL_DEV_TIMEOUT.  This call launches one 128-thread block that uses that same wait:
 * warp 0 waits on a barrier that completes, warps 1-3 on one that nobody arrives at, each
 * for at most poll_limit polls (1 .. 2^20).  The kernel always returns; afterwards
 * status_word has ZIPVL_DEV_TIMEOUT set and progress[0..4) (device int32, may be NULL)
 * holds 1 for the warp whose wait succeeded and 0 for the three that gave up.  The CUDA
 * context stays usable.
 */
zipvl_status zipvl_selftest_wait_timeout(int32_t poll_limit, int32_t *progress,
                                         int32_t *status_word, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* ZIPVL_H_ */
