"""ctypes binding of libzipvl.so -- argument marshalling only.

Each function has the name of the C entry point it calls (see include/zipvl.h)
and does nothing but turn torch tensors into pointers, allocate outputs the
caller did not pass (torch is used for device memory and streams only) and
raise ``ZipvlError`` on a non-zero status.  Every step of the path runs in the
library's CUDA kernels; there is no fallback: if the library cannot be loaded
the first call raises.
"""
import ctypes as C
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libzipvl.so")

ZIPVL_BF16, ZIPVL_F32, ZIPVL_F16 = 0, 1, 2
OP_SCORE, OP_SELECT, OP_SPARSE_PREFILL, OP_COMPACT_KV, OP_DECODE = range(5)
BUDGET_BY_NORM, TOPK_BY_ACC = 1, 2
OUT_PADDED, OUT_COMPACT = 0, 1
DEV_BAD_INDEX, DEV_TIMEOUT, DEV_CAPACITY, DEV_BAD_VALUE = 1, 2, 4, 8

EXPORTS = ["zipvl_status_string", "zipvl_last_error", "zipvl_version", "zipvl_launch_count",
           "zipvl_workspace_bytes",
           "zipvl_score", "zipvl_select", "zipvl_sparse_prefill", "zipvl_compact_kv",
           "zipvl_sparse_prefill_compact", "zipvl_workspace_bytes_batch", "zipvl_score_batch",
           "zipvl_select_batch", "zipvl_sparse_prefill_batch",
           "zipvl_decode", "zipvl_decode_paged", "zipvl_quantize_kv", "zipvl_decode_quant", "zipvl_decode_quant_batch", "zipvl_decode_noalloc", "zipvl_prefill_layer_host", "zipvl_layer_step_host",
           "zipvl_release_host_scratch", "zipvl_selftest_wait_timeout"]


class ZipvlError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"zipvl status {status}: {text}")
        self.status = status


class zipvl_layer(C.Structure):
    _fields_ = [("L", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("dtype", C.c_int32), ("reserved", C.c_int32),
                ("q_stride_tok", C.c_int64), ("kv_stride_tok", C.c_int64),
                ("softmax_scale", C.c_float), ("reserved2", C.c_int32)]


class zipvl_decode_desc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("dtype", C.c_int32), ("softmax_scale", C.c_float)]


class zipvl_batch(C.Structure):
    _fields_ = [("n_seq", C.c_int32), ("reserved", C.c_int32), ("q_stride_seq", C.c_int64),
                ("kv_stride_seq", C.c_int64)]


_lib = None


def load():
    """Load libzipvl.so (built in-tree by build.py).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2410_08584_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, u32, f32, sz = C.c_void_p, C.c_int32, C.c_uint32, C.c_float, C.c_size_t
    lp = C.POINTER(zipvl_layer)
    lib.zipvl_status_string.restype = C.c_char_p
    lib.zipvl_status_string.argtypes = [C.c_int]
    lib.zipvl_last_error.restype = C.c_char_p
    lib.zipvl_last_error.argtypes = []
    lib.zipvl_version.restype = i32
    lib.zipvl_launch_count.restype = C.c_uint64
    lib.zipvl_launch_count.argtypes = []
    lib.zipvl_workspace_bytes.restype = sz
    lib.zipvl_workspace_bytes.argtypes = [i32, lp, i32, i32]
    lib.zipvl_score.restype = C.c_int
    lib.zipvl_score.argtypes = [lp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp, vp]
    lib.zipvl_select.restype = C.c_int
    lib.zipvl_select.argtypes = [i32, vp, vp, f32, u32, i32, vp, vp, vp, vp, sz, vp, vp]
    lib.zipvl_sparse_prefill.restype = C.c_int
    lib.zipvl_sparse_prefill.argtypes = [lp, vp, vp, vp, vp, vp, i32, vp, i32, vp, sz, vp, vp]
    lib.zipvl_compact_kv.restype = C.c_int
    lib.zipvl_compact_kv.argtypes = [lp, vp, vp, vp, vp, i32, vp, vp, i32, vp, vp, vp]
    lib.zipvl_sparse_prefill_compact.restype = C.c_int
    lib.zipvl_sparse_prefill_compact.argtypes = [lp, vp, vp, vp, vp, vp, i32, vp, i32, vp, vp, i32, vp,
                                                 vp, sz, vp, vp]
    lib.zipvl_decode.restype = C.c_int
    lib.zipvl_decode.argtypes = [C.POINTER(zipvl_decode_desc), vp, vp, vp, vp, vp, vp, vp, vp,
                                 i32, vp, vp, sz, vp, vp]
    bp = C.POINTER(zipvl_batch)
    lib.zipvl_workspace_bytes_batch.restype = sz
    lib.zipvl_workspace_bytes_batch.argtypes = [i32, lp, i32, i32]
    lib.zipvl_score_batch.restype = C.c_int
    lib.zipvl_score_batch.argtypes = [lp, bp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp, vp]
    lib.zipvl_select_batch.restype = C.c_int
    lib.zipvl_select_batch.argtypes = [i32, i32, vp, vp, f32, u32, i32, vp, vp, vp, vp, sz, vp, vp]
    lib.zipvl_sparse_prefill_batch.restype = C.c_int
    lib.zipvl_sparse_prefill_batch.argtypes = [lp, bp, vp, vp, vp, vp, vp, i32, vp, i32, vp, vp, i32, vp,
                                               vp, sz, vp, vp]
    lib.zipvl_decode_paged.restype = C.c_int
    lib.zipvl_decode_paged.argtypes = [C.POINTER(zipvl_decode_desc), vp, vp, vp, vp, vp, vp, i32, i32, i32,
                                       vp, vp, i32, vp, vp, sz, vp, vp]
    lib.zipvl_quantize_kv.restype = C.c_int
    lib.zipvl_quantize_kv.argtypes = [lp, vp, vp, vp, vp, i32, vp, vp, vp, i32, vp, vp, vp, i32, vp, vp, vp]
    lib.zipvl_decode_quant.restype = C.c_int
    lib.zipvl_decode_quant.argtypes = [C.POINTER(zipvl_decode_desc), vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, i32,
                                       vp, i32, vp, vp, sz, vp, vp]
    lib.zipvl_decode_quant_batch.restype = C.c_int
    lib.zipvl_decode_quant_batch.argtypes = [C.POINTER(zipvl_decode_desc), vp, vp, vp, vp, i32, vp, vp, sz, vp, vp]
    lib.zipvl_decode_noalloc.restype = C.c_int
    lib.zipvl_decode_noalloc.argtypes = [C.POINTER(zipvl_decode_desc), vp, vp, vp, vp, vp, vp, vp,
                                         vp, i32, vp, vp, vp]
    lib.zipvl_prefill_layer_host.restype = C.c_int
    lib.zipvl_prefill_layer_host.argtypes = [lp, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp, vp]
    lib.zipvl_layer_step_host.restype = C.c_int
    lib.zipvl_layer_step_host.argtypes = [lp, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.zipvl_selftest_wait_timeout.restype = C.c_int
    lib.zipvl_selftest_wait_timeout.argtypes = [i32, vp, vp, vp]
    _lib = lib
    return lib


def _check(status):
    if status != 0:
        raise ZipvlError(status, load().zipvl_last_error().decode())


def _dtype_code(t):
    if t.dtype == torch.bfloat16:
        return ZIPVL_BF16
    if t.dtype == torch.float32:
        return ZIPVL_F32
    if t.dtype == torch.float16:
        return ZIPVL_F16
    raise TypeError(f"zipvl: dtype {t.dtype} (bfloat16, float16 or float32)")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _token_strided(t):
    """[L, H, d] with contiguous (H, d) rows and any token stride >= H*d (a slice of a fused
    QKV buffer, say): the layout the C ABI describes with q_stride_tok / kv_stride_tok."""
    return (t.dim() == 3 and t.stride(2) == 1 and t.stride(1) == t.shape[2]
            and t.stride(0) >= t.shape[1] * t.shape[2])


def _dev(t, name, dtype=None, token_strided=False):
    if not t.is_cuda or not (t.is_contiguous() or (token_strided and _token_strided(t))):
        raise ValueError(f"zipvl: {name} must be a contiguous CUDA tensor" +
                         (" (or [L, H, d] rows with a token stride)" if token_strided else ""))
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"zipvl: {name} must be {dtype}")
    return t


def _same_stride(k, v):
    if k.stride(0) != v.stride(0) or k.shape != v.shape:
        raise ValueError("zipvl: k and v must have the same shape and token stride")


def layer_desc(q, k, softmax_scale=0.0):
    """zipvl_layer for Q [L,Hq,d] and K [L,Hkv,d]: contiguous, or rows with a token stride
    (V must then have K's stride)."""
    L, Hq, d = q.shape
    qs = 0 if q.is_contiguous() else q.stride(0)
    ks = 0 if k.is_contiguous() else k.stride(0)
    return zipvl_layer(L, Hq, k.shape[1], d, _dtype_code(q), 0, qs, ks, float(softmax_scale), 0)


def zipvl_launch_count():
    return int(load().zipvl_launch_count())


def zipvl_workspace_bytes(op, layer, n_probe=0, batch=1):
    return int(load().zipvl_workspace_bytes(op, C.byref(layer), n_probe, batch))


def workspace(nbytes, device):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def zipvl_score(layer, q, k, probe_pos, acc=None, norm=None, total=None, ws=None, status=None,
                stream=None):
    """Probe attention scores: returns (acc float32[L], norm float32[L])."""
    _dev(q, "q", token_strided=True), _dev(k, "k", token_strided=True), _dev(probe_pos, "probe_pos", torch.int32)
    dev = q.device
    acc = torch.empty(layer.L, dtype=torch.float32, device=dev) if acc is None else acc
    norm = torch.empty(layer.L, dtype=torch.float32, device=dev) if norm is None else norm
    if ws is None:
        ws = workspace(zipvl_workspace_bytes(OP_SCORE, layer, probe_pos.numel()), dev)
    _check(load().zipvl_score(C.byref(layer), _ptr(q), _ptr(k), _ptr(probe_pos),
                              probe_pos.numel(), _ptr(acc), _ptr(norm), _ptr(total), _ptr(ws),
                              ws.numel(), _ptr(status), _stream(stream)))
    return acc, norm


def keep_last(r: int) -> int:
    """Mode bits of zipvl_select that add the last r positions to T (ZIPVL_KEEP_LAST)."""
    return int(r) << 8


def zipvl_select(acc, norm, tau, mode=0, fixed_k=0, k_out=None, idx=None, kept_mass=None,
                 ws=None, status=None, stream=None):
    """Budget and token set: returns (k_out int32[1], idx int32[L]) on the device."""
    _dev(acc, "acc", torch.float32), _dev(norm, "norm", torch.float32)
    L, dev = acc.numel(), acc.device
    k_out = torch.empty(1, dtype=torch.int32, device=dev) if k_out is None else k_out
    idx = torch.empty(L, dtype=torch.int32, device=dev) if idx is None else idx
    if ws is None:
        lay = zipvl_layer(L, 1, 1, 64, ZIPVL_F32, 0, 0, 0, 0.0, 0)
        ws = workspace(zipvl_workspace_bytes(OP_SELECT, lay), dev)
    _check(load().zipvl_select(L, _ptr(acc), _ptr(norm), float(tau), mode, fixed_k, _ptr(k_out),
                               _ptr(idx), _ptr(kept_mass), _ptr(ws), ws.numel(), _ptr(status),
                               _stream(stream)))
    return k_out, idx


def zipvl_sparse_prefill(layer, q, k, v, idx, k_dev, k_max, out=None, out_mode=OUT_PADDED,
                         ws=None, status=None, stream=None):
    """Causal attention over the kept tokens; returns out ([L,Hq,d] or [k_max,Hq,d])."""
    _dev(q, "q", token_strided=True), _dev(k, "k", token_strided=True), _dev(v, "v", token_strided=True), _dev(idx, "idx", torch.int32)
    _same_stride(k, v)
    _dev(k_dev, "k_dev", torch.int32)
    if out is None:
        rows = layer.L if out_mode == OUT_PADDED else k_max
        out = torch.empty((rows, layer.n_q_heads, layer.head_dim), dtype=q.dtype, device=q.device)
    if ws is None:
        ws = workspace(zipvl_workspace_bytes(OP_SPARSE_PREFILL, layer), q.device)
    _check(load().zipvl_sparse_prefill(C.byref(layer), _ptr(q), _ptr(k), _ptr(v), _ptr(idx),
                                       _ptr(k_dev), int(k_max), _ptr(out), out_mode, _ptr(ws),
                                       ws.numel(), _ptr(status), _stream(stream)))
    return out


def zipvl_sparse_prefill_compact(layer, q, k, v, idx, k_dev, k_max, k_cache, v_cache, capacity,
                                 out=None, out_mode=OUT_PADDED, len_out=None, ws=None, status=None,
                                 stream=None):
    """zipvl_sparse_prefill and zipvl_compact_kv in one call; returns (out, len_out)."""
    _dev(q, "q", token_strided=True), _dev(k, "k", token_strided=True), _dev(v, "v", token_strided=True), _dev(idx, "idx", torch.int32)
    _same_stride(k, v)
    _dev(k_dev, "k_dev", torch.int32), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache")
    if out is None:
        rows = layer.L if out_mode == OUT_PADDED else k_max
        out = torch.empty((rows, layer.n_q_heads, layer.head_dim), dtype=q.dtype, device=q.device)
    if ws is None:
        ws = workspace(zipvl_workspace_bytes(OP_SPARSE_PREFILL, layer), q.device)
    len_out = torch.empty(1, dtype=torch.int32, device=k.device) if len_out is None else len_out
    _check(load().zipvl_sparse_prefill_compact(
        C.byref(layer), _ptr(q), _ptr(k), _ptr(v), _ptr(idx), _ptr(k_dev), int(k_max), _ptr(out),
        out_mode, _ptr(k_cache), _ptr(v_cache), int(capacity), _ptr(len_out), _ptr(ws), ws.numel(),
        _ptr(status), _stream(stream)))
    return out, len_out


def _batch_desc(q, k):
    """zipvl_layer + zipvl_batch for stacked Q [n_seq, L, Hq, d] and K [n_seq, L, Hkv, d]
    (contiguous)."""
    if q.dim() != 4 or not q.is_contiguous() or not k.is_contiguous():
        raise ValueError("zipvl: batched calls take contiguous [n_seq, L, H, d] tensors")
    n_seq, L, Hq, d = q.shape
    lay = zipvl_layer(L, Hq, k.shape[2], d, _dtype_code(q), 0, 0, 0, 0.0, 0)
    return lay, zipvl_batch(n_seq, 0, 0, 0)


def zipvl_score_batch(q, k, probe_pos, acc=None, norm=None, ws=None, status=None, stream=None):
    """zipvl_score for stacked sequences: q [n_seq,L,Hq,d], k [n_seq,L,Hkv,d], probe_pos int32
    [n_seq,P]; returns (acc, norm) float32 [n_seq, L]."""
    _dev(q, "q"), _dev(k, "k"), _dev(probe_pos, "probe_pos", torch.int32)
    lay, b = _batch_desc(q, k)
    n_seq, L, P = q.shape[0], q.shape[1], probe_pos.shape[1]
    acc = torch.empty(n_seq, L, dtype=torch.float32, device=q.device) if acc is None else acc
    norm = torch.empty(n_seq, L, dtype=torch.float32, device=q.device) if norm is None else norm
    if ws is None:
        ws = workspace(load().zipvl_workspace_bytes_batch(OP_SCORE, C.byref(lay), P, n_seq), q.device)
    _check(load().zipvl_score_batch(C.byref(lay), C.byref(b), _ptr(q), _ptr(k), _ptr(probe_pos), P, _ptr(acc),
                                    _ptr(norm), None, _ptr(ws), ws.numel(), _ptr(status), _stream(stream)))
    return acc, norm


def zipvl_select_batch(acc, norm, tau, mode=0, fixed_k=0, k_out=None, idx=None, ws=None, status=None,
                       stream=None):
    """zipvl_select for score rows [n_seq, L]; returns (k_out int32[n_seq], idx int32[n_seq, L])."""
    _dev(acc, "acc", torch.float32), _dev(norm, "norm", torch.float32)
    n_seq, L = acc.shape
    k_out = torch.empty(n_seq, dtype=torch.int32, device=acc.device) if k_out is None else k_out
    idx = torch.empty(n_seq, L, dtype=torch.int32, device=acc.device) if idx is None else idx
    if ws is None:
        lay = zipvl_layer(L, 1, 1, 64, ZIPVL_F32, 0, 0, 0, 0.0, 0)
        ws = workspace(zipvl_workspace_bytes(OP_SELECT, lay), acc.device)
    _check(load().zipvl_select_batch(L, n_seq, _ptr(acc), _ptr(norm), float(tau), mode, fixed_k, _ptr(k_out),
                                     _ptr(idx), None, _ptr(ws), ws.numel(), _ptr(status), _stream(stream)))
    return k_out, idx


def zipvl_sparse_prefill_batch(q, k, v, idx, k_dev, k_max, k_cache=None, v_cache=None, capacity=0, out=None,
                               out_mode=OUT_PADDED, len_out=None, ws=None, status=None, stream=None):
    """zipvl_sparse_prefill (and, with caches, zipvl_compact_kv) for stacked sequences; returns
    (out [n_seq, L or k_max, Hq, d], len_out or None)."""
    _dev(q, "q"), _dev(k, "k"), _dev(v, "v"), _dev(idx, "idx", torch.int32), _dev(k_dev, "k_dev", torch.int32)
    lay, b = _batch_desc(q, k)
    n_seq, L = q.shape[0], q.shape[1]
    if out is None:
        rows = L if out_mode == OUT_PADDED else k_max
        out = torch.empty((n_seq, rows, lay.n_q_heads, lay.head_dim), dtype=q.dtype, device=q.device)
    if ws is None:
        ws = workspace(zipvl_workspace_bytes(OP_SPARSE_PREFILL, lay), q.device)
    if k_cache is not None and len_out is None:
        len_out = torch.empty(n_seq, dtype=torch.int32, device=q.device)
    _check(load().zipvl_sparse_prefill_batch(C.byref(lay), C.byref(b), _ptr(q), _ptr(k), _ptr(v), _ptr(idx),
                                             _ptr(k_dev), int(k_max), _ptr(out), out_mode, _ptr(k_cache),
                                             _ptr(v_cache), int(capacity), _ptr(len_out), _ptr(ws), ws.numel(),
                                             _ptr(status), _stream(stream)))
    return out, len_out


def zipvl_release_host_scratch():
    """Return the device memory zipvl_prefill_layer_host keeps between calls."""
    lib = load()
    lib.zipvl_release_host_scratch.restype = C.c_int
    _check(lib.zipvl_release_host_scratch())


def zipvl_compact_kv(layer, k, v, idx, k_dev, k_max, k_cache, v_cache, capacity, len_out=None,
                     status=None, stream=None):
    """K = K[T], V = V[T] into caller-owned caches; returns len_out int32[1]."""
    _dev(k, "k", token_strided=True), _dev(v, "v", token_strided=True), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache")
    _same_stride(k, v)
    len_out = torch.empty(1, dtype=torch.int32, device=k.device) if len_out is None else len_out
    _check(load().zipvl_compact_kv(C.byref(layer), _ptr(k), _ptr(v), _ptr(idx), _ptr(k_dev),
                                   int(k_max), _ptr(k_cache), _ptr(v_cache), int(capacity),
                                   _ptr(len_out), _ptr(status), _stream(stream)))
    return len_out


def zipvl_decode(desc, q, k_new, v_new, k_cache, v_cache, cache_off, capacity, seq_lens, max_len,
                 out=None, ws=None, status=None, stream=None):
    """One decode step over the ragged batch of caches; returns out [B,Hq,d]."""
    _dev(q, "q"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache")
    _dev(cache_off, "cache_off", torch.int64), _dev(capacity, "capacity", torch.int32)
    _dev(seq_lens, "seq_lens", torch.int32)
    out = torch.empty_like(q) if out is None else out
    if ws is None:
        lay = zipvl_layer(int(max_len), desc.n_q_heads, desc.n_kv_heads, desc.head_dim, desc.dtype,
                          0, 0, 0, 0.0, 0)
        ws = workspace(zipvl_workspace_bytes(OP_DECODE, lay, 0, desc.batch), q.device)
    _check(load().zipvl_decode(C.byref(desc), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                               _ptr(v_cache), _ptr(cache_off), _ptr(capacity), _ptr(seq_lens),
                               int(max_len), _ptr(out), _ptr(ws), ws.numel(), _ptr(status),
                               _stream(stream)))
    return out


def zipvl_decode_paged(desc, q, k_new, v_new, k_pages, v_pages, block_table, capacity, seq_lens, max_len,
                       out=None, ws=None, status=None, stream=None):
    """One decode step over paged caches: k_pages / v_pages [n_pages, page_rows, Hkv, d],
    block_table int32 [B, max_pages]; returns out [B,Hq,d]."""
    _dev(q, "q"), _dev(k_pages, "k_pages"), _dev(v_pages, "v_pages")
    _dev(block_table, "block_table", torch.int32), _dev(capacity, "capacity", torch.int32)
    _dev(seq_lens, "seq_lens", torch.int32)
    out = torch.empty_like(q) if out is None else out
    if ws is None:
        lay = zipvl_layer(int(max_len), desc.n_q_heads, desc.n_kv_heads, desc.head_dim, desc.dtype,
                          0, 0, 0, 0.0, 0)
        ws = workspace(zipvl_workspace_bytes(OP_DECODE, lay, 0, desc.batch), q.device)
    _check(load().zipvl_decode_paged(C.byref(desc), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_pages),
                                     _ptr(v_pages), _ptr(block_table), block_table.shape[1],
                                     k_pages.shape[1], k_pages.shape[0], _ptr(capacity), _ptr(seq_lens),
                                     int(max_len), _ptr(out), _ptr(ws), ws.numel(), _ptr(status),
                                     _stream(stream)))
    return out


class QuantCache:
    """Device buffers of one sequence's mixed-precision cache (see zipvl_quantize_kv in
    include/zipvl.h): 4-bit block for the tokens of T plus room for `extra` decoded tokens,
    2-bit block for the others."""

    def __init__(self, L, n_kv_heads, head_dim, dtype, device, cap_hi, cap_lo):
        u8 = torch.uint8
        self.cap_hi, self.cap_lo = int(cap_hi), int(cap_lo)
        self.k_hi = torch.zeros(self.cap_hi, n_kv_heads, head_dim // 2, dtype=u8, device=device)
        self.v_hi = torch.zeros_like(self.k_hi)
        self.p_hi = torch.zeros(self.cap_hi, n_kv_heads, 4, dtype=dtype, device=device)
        self.k_lo = torch.zeros(self.cap_lo, n_kv_heads, head_dim // 4, dtype=u8, device=device)
        self.v_lo = torch.zeros_like(self.k_lo)
        self.p_lo = torch.zeros(self.cap_lo, n_kv_heads, 4, dtype=dtype, device=device)
        self.lens = torch.zeros(2, dtype=torch.int32, device=device)

    def nbytes(self, n_hi, n_lo):
        """Bytes the first n_hi / n_lo rows of the blocks take (codes of K and V + parameters)."""
        per_hi = 2 * self.k_hi[0].numel() + self.p_hi[0].numel() * self.p_hi.element_size()
        per_lo = 2 * self.k_lo[0].numel() + self.p_lo[0].numel() * self.p_lo.element_size()
        return n_hi * per_hi + n_lo * per_lo


def zipvl_quantize_kv(layer, k, v, idx, k_dev, k_max, cache, status=None, stream=None):
    """K, V and the token set into the mixed-precision cache; returns cache.lens (device int32[2])."""
    _dev(k, "k", token_strided=True), _dev(v, "v", token_strided=True), _dev(idx, "idx", torch.int32)
    _same_stride(k, v)
    _check(load().zipvl_quantize_kv(C.byref(layer), _ptr(k), _ptr(v), _ptr(idx), _ptr(k_dev), int(k_max),
                                    _ptr(cache.k_hi), _ptr(cache.v_hi), _ptr(cache.p_hi), cache.cap_hi,
                                    _ptr(cache.k_lo), _ptr(cache.v_lo), _ptr(cache.p_lo), cache.cap_lo,
                                    _ptr(cache.lens), _ptr(status), _stream(stream)))
    return cache.lens


def zipvl_decode_quant(desc, q, k_new, v_new, cache, max_len, out=None, ws=None, status=None, stream=None):
    """One decode step of one request over its mixed-precision cache; returns out [1,Hq,d]."""
    _dev(q, "q")
    out = torch.empty_like(q) if out is None else out
    if ws is None:
        lay = zipvl_layer(int(max_len), desc.n_q_heads, desc.n_kv_heads, desc.head_dim, desc.dtype,
                          0, 0, 0, 0.0, 0)
        ws = workspace(zipvl_workspace_bytes(OP_DECODE, lay, 0, 1), q.device)
    _check(load().zipvl_decode_quant(C.byref(desc), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(cache.k_hi),
                                     _ptr(cache.v_hi), _ptr(cache.p_hi), cache.cap_hi, _ptr(cache.k_lo),
                                     _ptr(cache.v_lo), _ptr(cache.p_lo), cache.cap_lo, _ptr(cache.lens),
                                     int(max_len), _ptr(out), _ptr(ws), ws.numel(), _ptr(status),
                                     _stream(stream)))
    return out


def quant_cache_table(caches, device):
    """The device table zipvl_decode_quant_batch takes: one 64-byte zipvl_quant_cache entry per
    request (seven device pointers, then the two capacities)."""
    rows = []
    for c in caches:
        rows.append([c.k_hi.data_ptr(), c.v_hi.data_ptr(), c.p_hi.data_ptr(), c.k_lo.data_ptr(),
                     c.v_lo.data_ptr(), c.p_lo.data_ptr(), c.lens.data_ptr(),
                     (int(c.cap_hi) & 0xffffffff) | (int(c.cap_lo) << 32)])
    return torch.tensor(rows, dtype=torch.int64).to(device)


def zipvl_decode_quant_batch(desc, q, k_new, v_new, table, max_len, out=None, ws=None, status=None, stream=None):
    """One decode step of desc.batch requests over their mixed-precision caches (table:
    quant_cache_table of the requests' QuantCache objects); returns out [B,Hq,d]."""
    _dev(q, "q"), _dev(table, "table", torch.int64)
    if table.shape[0] != desc.batch or table.shape[1] != 8:
        raise ValueError("table must be int64 [batch, 8]")
    out = torch.empty_like(q) if out is None else out
    if ws is None:
        lay = zipvl_layer(int(max_len), desc.n_q_heads, desc.n_kv_heads, desc.head_dim, desc.dtype,
                          0, 0, 0, 0.0, 0)
        ws = workspace(zipvl_workspace_bytes(OP_DECODE, lay, 0, desc.batch), q.device)
    _check(load().zipvl_decode_quant_batch(C.byref(desc), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(table),
                                           int(max_len), _ptr(out), _ptr(ws), ws.numel(), _ptr(status),
                                           _stream(stream)))
    return out


def zipvl_decode_noalloc(desc, q, k_new, v_new, k_cache, v_cache, cache_off, capacity, seq_lens,
                         max_len, out, status=None, stream=None):
    """zipvl_decode for callers that cannot allocate: the scratch is a fixed
    array inside the library, and this wrapper allocates nothing either (the
    caller passes `out`).  Raises ZipvlError (workspace) beyond the 8 MiB limit."""
    _dev(q, "q"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"), _dev(out, "out")
    _dev(cache_off, "cache_off", torch.int64), _dev(capacity, "capacity", torch.int32)
    _dev(seq_lens, "seq_lens", torch.int32)
    _check(load().zipvl_decode_noalloc(C.byref(desc), _ptr(q), _ptr(k_new), _ptr(v_new),
                                       _ptr(k_cache), _ptr(v_cache), _ptr(cache_off),
                                       _ptr(capacity), _ptr(seq_lens), int(max_len), _ptr(out),
                                       _ptr(status), _stream(stream)))
    return out


def zipvl_selftest_wait_timeout(poll_limit, progress, status, stream=None):
    """Launch the library's bounded-wait self-test (see include/zipvl.h)."""
    _dev(progress, "progress", torch.int32), _dev(status, "status", torch.int32)
    _check(load().zipvl_selftest_wait_timeout(int(poll_limit), _ptr(progress), _ptr(status),
                                              _stream(stream)))


def zipvl_layer_step_host(layer, q, k, v, probe_pos, tau, q_new, k_new, v_new, out=None, k_cache=None,
                          v_cache=None, idx=None, decode_out=None):
    """Algorithm 1 for the layer and one decode step (Algorithm 2) on the cache it leaves,
    from HOST tensors.  Returns (k, idx, out, k_cache, v_cache, decode_out) as host tensors."""
    for t in (q, k, v, probe_pos, q_new, k_new, v_new):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("zipvl_layer_step_host takes contiguous host tensors")
    pin = q.is_pinned()
    mk = lambda shape, dt: torch.empty(shape, dtype=dt, pin_memory=pin)
    out = mk(q.shape, q.dtype) if out is None else out
    k_cache = mk(k.shape, k.dtype) if k_cache is None else k_cache
    v_cache = mk(v.shape, v.dtype) if v_cache is None else v_cache
    idx = mk((layer.L,), torch.int32) if idx is None else idx
    decode_out = mk(q_new.shape, q_new.dtype) if decode_out is None else decode_out
    kk = C.c_int32(0)
    _check(load().zipvl_layer_step_host(C.byref(layer), _ptr(q), _ptr(k), _ptr(v), _ptr(probe_pos),
                                        probe_pos.numel(), float(tau), C.cast(C.byref(kk), C.c_void_p),
                                        _ptr(idx), _ptr(out), _ptr(k_cache), _ptr(v_cache), _ptr(q_new),
                                        _ptr(k_new), _ptr(v_new), _ptr(decode_out)))
    return kk.value, idx, out, k_cache, v_cache, decode_out


def zipvl_prefill_layer_host(layer, q, k, v, probe_pos, tau, out=None, k_cache=None, v_cache=None,
                             idx=None):
    """Algorithm 1 end to end from HOST tensors (copies in, runs, copies back).
    Returns (k, idx, out, k_cache, v_cache) as host tensors."""
    for t in (q, k, v, probe_pos):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("zipvl_prefill_layer_host takes contiguous host tensors")
    pin = q.is_pinned()
    mk = lambda shape, dt: torch.empty(shape, dtype=dt, pin_memory=pin)
    out = mk(q.shape, q.dtype) if out is None else out
    k_cache = mk(k.shape, k.dtype) if k_cache is None else k_cache
    v_cache = mk(v.shape, v.dtype) if v_cache is None else v_cache
    idx = mk((layer.L,), torch.int32) if idx is None else idx
    kk = C.c_int32(0)
    _check(load().zipvl_prefill_layer_host(C.byref(layer), _ptr(q), _ptr(k), _ptr(v),
                                           _ptr(probe_pos), probe_pos.numel(), float(tau),
                                           C.cast(C.byref(kk), C.c_void_p), _ptr(idx), _ptr(out),
                                           _ptr(k_cache), _ptr(v_cache)))
    return kk.value, idx, out, k_cache, v_cache
