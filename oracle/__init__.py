"""CPU oracle for the ZipVL per-layer hot path -- TEST INFRASTRUCTURE ONLY.

numpy front end of ``zipvl_oracle.c`` (fp64, plain loops, OpenMP over heads).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library never does, and nothing here imports it.

Every function names the passage of the paper it follows.  Inputs are numpy
arrays holding the stored values exactly (bf16 tensors are passed upcast to
float32, which is lossless); results are float64 / int32.
"""
import ctypes as C
import math

import numpy as np

from .build import build as _build

_lib = None

_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")
_i64p = np.ctypeslib.ndpointer(np.int64, flags="C_CONTIGUOUS")
_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build())
        L.zo_probe_scores.restype = C.c_int
        L.zo_probe_scores.argtypes = [_f32p, _f32p, C.c_int, C.c_int, C.c_int, C.c_int, _i32p,
                                      C.c_int, C.c_double, _f64p, C.POINTER(C.c_double)]
        L.zo_normalise.restype = None
        L.zo_normalise.argtypes = [_f64p, C.c_int, _i32p, C.c_int, C.c_int, _f64p, _i32p]
        L.zo_budget.restype = C.c_int
        L.zo_budget.argtypes = [_f64p, C.c_int, C.c_double, _f64p]
        L.zo_topk_index.restype = None
        L.zo_topk_index.argtypes = [_f64p, C.c_int, C.c_int, _i32p]
        L.zo_sparse_prefill.restype = C.c_int
        L.zo_sparse_prefill.argtypes = [_f32p, _f32p, _f32p, C.c_int, C.c_int, C.c_int, C.c_int,
                                        _i32p, C.c_int, C.c_double, C.c_void_p, C.c_int, _f64p]
        L.zo_compact_rows.restype = None
        L.zo_compact_rows.argtypes = [_u8p, C.c_size_t, _i32p, C.c_int, _u8p]
        L.zo_decode.restype = None
        L.zo_decode.argtypes = [_f32p, C.c_void_p, C.c_void_p, _f32p, _f32p, _i64p, _i32p,
                                C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, _f64p]
        L.zo_threads.restype = C.c_int
        _lib = L
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle's parallel loops will use."""
    return int(lib().zo_threads())


def _f32(x):
    return np.ascontiguousarray(x, dtype=np.float32)


def _i32(x):
    return np.ascontiguousarray(x, dtype=np.int32)


def default_scale(d: int) -> float:
    """Softmax scale 1/sqrt(head_dim) (Eq. A writes sqrt(d_k))."""
    return 1.0 / math.sqrt(d)


def probe_scores(Q, K, probe_pos, scale=None):
    """Eq. A under the causal mask of Eq. 2, column-summed as in Eq. 6.

    Q [L,Hq,d], K [L,Hkv,d], probe_pos int[P].  Returns (acc float64[L], S)."""
    Q, K, probe_pos = _f32(Q), _f32(K), _i32(probe_pos)
    L, Hq, d = Q.shape
    Hkv = K.shape[1]
    assert K.shape == (L, Hkv, d)
    acc = np.zeros(L, np.float64)
    S = C.c_double(0.0)
    rc = lib().zo_probe_scores(Q, K, L, Hq, Hkv, d, probe_pos, len(probe_pos),
                               default_scale(d) if scale is None else float(scale),
                               acc, C.byref(S))
    if rc != 0:
        raise ValueError("zo_probe_scores: bad argument")
    return acc, S.value


def normalise(acc, probe_pos, n_q_heads):
    """Eq. 8 with the structural nnz.  Returns (norm float64[L], nnz int32[L])."""
    acc = np.ascontiguousarray(acc, np.float64)
    probe_pos = _i32(probe_pos)
    norm = np.zeros_like(acc)
    nnz = np.zeros(len(acc), np.int32)
    lib().zo_normalise(acc, len(acc), probe_pos, len(probe_pos), int(n_q_heads), norm, nnz)
    return norm, nnz


def budget(metric, tau):
    """Eq. 7.  Returns (p, diag) with diag = dict(S, C_prev, C_p, target)."""
    metric = np.ascontiguousarray(metric, np.float64)
    diag = np.zeros(4, np.float64)
    p = lib().zo_budget(metric, len(metric), float(tau), diag)
    return int(p), dict(S=diag[0], C_prev=diag[1], C_p=diag[2], target=diag[3])


def topk_index(metric, p):
    """Eq. 9, ties toward the smaller index, result ascending by position."""
    metric = np.ascontiguousarray(metric, np.float64)
    T = np.zeros(int(p), np.int32)
    lib().zo_topk_index(metric, len(metric), int(p), T)
    return T


METRIC_ACC, METRIC_NORM = 0, 1


def select(acc, norm, tau, budget_metric=METRIC_ACC, topk_metric=METRIC_NORM, fixed_k=0, keep_last=0):
    """Eq. 7 then Eq. 9: the accumulated score fixes p, the normalised score
    picks T (the paper's default pairing; Table B's other pairings by flag).
    fixed_k > 0 replaces the adaptive budget (the fixed-ratio ablation).
    keep_last = r > 0 (an option outside the paper, which does not say whether the
    final positions -- whose outputs produce the first generated token -- must
    survive): T becomes the union of Eq. 9's set and the last r positions, and the
    first value returned is the size of that union."""
    bm = acc if budget_metric == METRIC_ACC else norm
    tm = acc if topk_metric == METRIC_ACC else norm
    if fixed_k > 0:
        p, diag = min(int(fixed_k), len(bm)), {}
    else:
        p, diag = budget(bm, tau)
    T = topk_index(tm, p)
    if keep_last > 0:
        L = len(bm)
        T = np.union1d(T, np.arange(max(0, L - int(keep_last)), L)).astype(np.int32)
        p = len(T)
    return p, T, diag


def sparse_prefill(Q, K, V, T, scale=None, rows=None):
    """Algorithm 1's sparse attention: causal softmax attention (Eq. 2) over
    the gathered tokens Q[T], K[T], V[T].  Returns float64 [n_rows, Hq, d] for
    the listed rows of T (all p rows if rows is None)."""
    Q, K, V, T = _f32(Q), _f32(K), _f32(V), _i32(T)
    L, Hq, d = Q.shape
    Hkv = K.shape[1]
    if rows is None:
        n_rows, rows_p = len(T), None
    else:
        rows = _i32(rows)
        assert rows.size == 0 or (rows.min() >= 0 and rows.max() < len(T))
        n_rows, rows_p = len(rows), rows.ctypes.data
    out = np.zeros((n_rows, Hq, d), np.float64)
    rc = lib().zo_sparse_prefill(Q, K, V, L, Hq, Hkv, d, T, len(T),
                                 default_scale(d) if scale is None else float(scale),
                                 rows_p, n_rows, out)
    if rc != 0:
        raise ValueError("zo_sparse_prefill: bad argument")
    return out


def pad_rows(out_compact, T, L):
    """Outputs of tokens outside T are padded with zeros (Sec. 3.2)."""
    full = np.zeros((L,) + out_compact.shape[1:], out_compact.dtype)
    full[np.asarray(T)] = out_compact
    return full


def compact_rows(x, T):
    """Algorithm 1's cache step, x[T] copied byte for byte.  x is any
    C-contiguous array whose first axis is the token axis."""
    x = np.ascontiguousarray(x)
    T = _i32(T)
    row_bytes = x.strides[0]
    src = x.view(np.uint8).reshape(x.shape[0], row_bytes) if x.shape[0] else x.view(np.uint8)
    dst = np.zeros((len(T), row_bytes), np.uint8)
    lib().zo_compact_rows(src.reshape(-1), row_bytes, T, len(T), dst.reshape(-1))
    return dst.reshape(-1).view(x.dtype).reshape((len(T),) + x.shape[1:])


def decode_step(q, k_new, v_new, k_cache, v_cache, cache_off, seq_lens, n_kv_heads, scale=None):
    """Algorithm 2 (Eq. 4-5) for a ragged batch.  k_cache / v_cache are flat
    float32 arrays updated in place; seq_lens (int32[B]) is incremented when
    k_new / v_new are given.  Returns float64 [B, Hq, d]."""
    q = _f32(q)
    B, Hq, d = q.shape
    assert k_cache.dtype == np.float32 and k_cache.flags.c_contiguous
    assert v_cache.dtype == np.float32 and v_cache.flags.c_contiguous
    assert seq_lens.dtype == np.int32
    cache_off = np.ascontiguousarray(cache_off, np.int64)
    out = np.zeros((B, Hq, d), np.float64)
    if k_new is not None:
        k_new, v_new = _f32(k_new), _f32(v_new)
        kp, vp = k_new.ctypes.data, v_new.ctypes.data
    else:
        kp = vp = None
    lib().zo_decode(q, kp, vp, k_cache.reshape(-1), v_cache.reshape(-1), cache_off, seq_lens,
                    B, Hq, int(n_kv_heads), d,
                    default_scale(d) if scale is None else float(scale), out)
    return out


def decode_step_paged(q, k_new, v_new, k_pages, v_pages, block_table, seq_lens, scale=None):
    """Algorithm 2 (Eq. 4-5) where each request's cache is a list of pages of a shared pool: a
    storage layout, not a change of the method.  k_pages / v_pages are float32
    [n_pages, page_rows, Hkv, d] updated in place; block_table int32 [B, max_pages] names, in
    order, the pages that hold request b's rows.  Each request's rows are gathered into a
    contiguous cache, decode_step runs on those, and the appended rows are written back to the
    page they belong to.  Returns float64 [B, Hq, d]."""
    q = _f32(q)
    B = q.shape[0]
    n_pages, page_rows, Hkv, d = k_pages.shape
    block_table = np.asarray(block_table, np.int64)
    row = Hkv * d
    cap = block_table.shape[1] * page_rows
    kc = np.zeros((B, cap, Hkv, d), np.float32)
    vc = np.zeros_like(kc)
    for b in range(B):
        n_used = -(-(int(seq_lens[b]) + 1) // page_rows)          # pages that hold rows, with room for one more
        for i in range(min(n_used, block_table.shape[1])):
            kc[b, i * page_rows:(i + 1) * page_rows] = k_pages[block_table[b, i]]
            vc[b, i * page_rows:(i + 1) * page_rows] = v_pages[block_table[b, i]]
    off = (np.arange(B, dtype=np.int64) * cap * row)
    old = np.array(seq_lens, np.int32).copy()
    out = decode_step(q, k_new, v_new, kc.reshape(-1), vc.reshape(-1), off, seq_lens, Hkv, scale)
    if k_new is not None:
        for b in range(B):
            r = int(old[b])
            if int(seq_lens[b]) == r + 1:                          # the row was appended
                page = block_table[b, r // page_rows]
                k_pages[page, r % page_rows] = kc[b, r]
                v_pages[page, r % page_rows] = vc[b, r]
    return out


# ---------------------------------------------------------------------------------------
# Mixed-precision KV cache (Sec. 4.3, Table 3: "important tokens are quantized to 4-bit,
# while other tokens are quantized to 2-bit").  The paper takes the quantiser from the work
# it cites and only fixes the bit allocation; the reading used here: every token stays in
# the cache; keys and values are quantised per (token, KV head) over the head_dim channels
# with an asymmetric uniform quantiser whose scale and zero point are kept in the storage
# type; the codes are decided in fp32 (the precision the kernel takes that decision in).
# ---------------------------------------------------------------------------------------
def _round_to_storage(x, storage):
    """fp32 values rounded (to nearest even) to the storage type, returned as fp32."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, np.float32))
    if storage == "bf16":
        return t.to(torch.bfloat16).float().numpy()
    if storage == "f16":
        return t.to(torch.float16).float().numpy()
    return t.numpy().copy()


def quantize_rows(x, bits, storage="bf16"):
    """x float32 [n, H, d] (stored values).  Per (row, head): lo = min, hi = max over the d
    channels, scale = (hi - lo) / (2^bits - 1) in fp32; scale and lo are rounded to the
    storage type; inv = 1 / scale; code_c = clip(rint((x_c - lo) * inv), 0, 2^bits - 1), every
    step one fp32 operation (one division per row, a subtraction and a multiplication per value).
    A row of equal values (scale 0) gets codes 0.  Returns (codes uint8 [n,H,d],
    scale float32 [n,H], zero float32 [n,H])."""
    x = np.ascontiguousarray(x, np.float32)
    levels = np.float32((1 << bits) - 1)
    lo = x.min(axis=-1)
    hi = x.max(axis=-1)
    scale = _round_to_storage((hi - lo).astype(np.float32) / levels, storage)
    zero = _round_to_storage(lo, storage)
    safe = np.where(scale > 0, scale, np.float32(1.0)).astype(np.float32)
    inv = (np.float32(1.0) / safe).astype(np.float32)
    qf = np.rint(((x - zero[..., None]).astype(np.float32) * inv[..., None]).astype(np.float32))
    codes = np.clip(qf, 0, levels).astype(np.uint8)
    codes[scale <= 0] = 0
    return codes, scale.astype(np.float32), zero.astype(np.float32)


def dequantize_rows(codes, scale, zero):
    """x^ = code * scale + zero, in float64."""
    return codes.astype(np.float64) * scale.astype(np.float64)[..., None] + zero.astype(np.float64)[..., None]


def pack_codes(codes, bits):
    """Codes of `bits` bits packed little-end first: channel c of a row sits in byte
    c * bits // 8 at bit offset (c * bits) % 8.  codes uint8 [..., d] -> uint8 [..., d*bits/8]."""
    codes = np.ascontiguousarray(codes, np.uint8)
    per = 8 // bits
    d = codes.shape[-1]
    assert d % per == 0
    g = codes.reshape(codes.shape[:-1] + (d // per, per)).astype(np.uint16)
    out = np.zeros(g.shape[:-1], np.uint16)
    for i in range(per):
        out |= g[..., i] << (bits * i)
    return out.astype(np.uint8)


def quantize_kv(K, V, T, storage="bf16", bits_hi=4, bits_lo=2):
    """The cache of one layer after Algorithm 1 when nothing is evicted but the precision
    follows the token set: the tokens of T (ascending) at bits_hi bits, the others
    (ascending) at bits_lo bits.  K, V float32 [L, Hkv, d].  Returns a dict with, for
    block in ("hi", "lo"): tokens (positions), k_codes, v_codes (uint8 [n,Hkv,d]), k_scale,
    k_zero, v_scale, v_zero (float32 [n,Hkv])."""
    K, V = _f32(K), _f32(V)
    T = np.asarray(T, np.int64)
    U = np.setdiff1d(np.arange(K.shape[0]), T)
    cache = {}
    for name, toks, bits in (("hi", T, bits_hi), ("lo", U, bits_lo)):
        kc, ks, kz = quantize_rows(K[toks], bits, storage)
        vc, vs, vz = quantize_rows(V[toks], bits, storage)
        cache[name] = dict(tokens=toks, bits=bits, k_codes=kc, v_codes=vc, k_scale=ks, k_zero=kz,
                           v_scale=vs, v_zero=vz)
    return cache


def decode_step_quant(q, k_new, v_new, cache, n_kv_heads, storage="bf16", scale=None):
    """Algorithm 2 (Eq. 4-5) over the mixed-precision cache of one request: the new key and
    value (float32 [1,Hkv,d], or None) are quantised at the high precision and appended to
    the "hi" block (Eq. 4); the query (float32 [1,Hq,d]) attends over the dequantised rows of
    both blocks (Eq. 5; softmax attention does not depend on the order of the cached rows).
    The cache dict is updated in place.  Returns float64 [1, Hq, d]."""
    hi, lo = cache["hi"], cache["lo"]
    if k_new is not None:
        kc, ks, kz = quantize_rows(_f32(k_new), hi["bits"], storage)
        vc, vs, vz = quantize_rows(_f32(v_new), hi["bits"], storage)
        for key, val in (("k_codes", kc), ("v_codes", vc), ("k_scale", ks), ("k_zero", kz),
                         ("v_scale", vs), ("v_zero", vz)):
            hi[key] = np.concatenate([hi[key], val])
        hi["tokens"] = np.concatenate([hi["tokens"], [-1]])
    kd = np.concatenate([dequantize_rows(b["k_codes"], b["k_scale"], b["k_zero"]) for b in (hi, lo)])
    vd = np.concatenate([dequantize_rows(b["v_codes"], b["v_scale"], b["v_zero"]) for b in (hi, lo)])
    n = kd.shape[0]
    # the dequantised rows are fp64; decode_step takes float32 caches, so the attention over
    # them is written out here directly, in float64
    q = np.asarray(q, np.float64)
    _, Hq, d = q.shape
    G = Hq // n_kv_heads
    sc = default_scale(d) if scale is None else float(scale)
    out = np.zeros((1, Hq, d), np.float64)
    for h in range(Hq):
        g = h // G
        if n == 0:
            continue
        s = sc * (kd[:, g, :] @ q[0, h])
        w = np.exp(s - s.max())
        w /= w.sum()
        out[0, h] = w @ vd[:, g, :]
    return out
