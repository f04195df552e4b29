"""GPU parity of the mixed-precision KV cache (Sec. 4.3, Table 3: tokens of T at 4 bits, the
others at 2) against the CPU oracle: codes, parameters and packing bit for bit; decode steps
over the quantised cache within the attention tolerance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_08584_b200 import workloads as W
from parity import check_attention, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _blocks_from_gpu(cache, n_hi, n_lo):
    f = lambda t: t.cpu().numpy()
    return dict(hi=dict(k=f(cache.k_hi[:n_hi]), v=f(cache.v_hi[:n_hi]), p=to_np(cache.p_hi[:n_hi])),
                lo=dict(k=f(cache.k_lo[:n_lo]), v=f(cache.v_lo[:n_lo]), p=to_np(cache.p_lo[:n_lo])))


def _check_blocks(got, ref):
    for name in ("hi", "lo"):
        b, bits = ref[name], ref[name]["bits"]
        n = len(b["tokens"])
        assert np.array_equal(got[name]["k"][:n], oracle.pack_codes(b["k_codes"], bits)), f"{name}: K codes"
        assert np.array_equal(got[name]["v"][:n], oracle.pack_codes(b["v_codes"], bits)), f"{name}: V codes"
        want_p = np.stack([b["k_scale"], b["k_zero"], b["v_scale"], b["v_zero"]], axis=-1)
        assert np.array_equal(got[name]["p"][:n], want_p), f"{name}: parameters"


@pytest.mark.parametrize("case", ["bf16_mha_d128", "fp16_gqa2_d128", "bf16_gqa4_d64", "bf16_ragged"])
def test_quantised_cache_and_decode_parity(zipvl, case):
    z = zipvl
    if case == "bf16_mha_d128":
        layer = W.heavy_key_layer(L_visual=1150, L_text=64, H=8, seed=81)
    elif case == "fp16_gqa2_d128":
        layer = W.heavy_key_layer(L_visual=700, L_text=33, H=8, Hkv=4, seed=82, dtype=torch.float16)
    elif case == "bf16_gqa4_d64":
        layer = W.heavy_key_layer(L_visual=500, L_text=41, H=8, Hkv=2, d=64, seed=83)
    else:
        layer = W.heavy_key_layer(L_visual=100, L_text=29, H=3, Hkv=3, seed=84)
    storage = "f16" if layer.q.dtype == torch.float16 else "bf16"
    L, Hq, Hkv, d = layer.L, layer.n_q_heads, layer.n_kv_heads, layer.head_dim
    q, k, v, probe = (t.to(DEV) for t in (layer.q, layer.k, layer.v, layer.probe_pos))
    desc = z.layer_desc(q, k)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    acc, norm = z.zipvl_score(desc, q, k, probe, status=st)
    k_dev, idx = z.zipvl_select(acc, norm, layer.tau, status=st)
    kk = int(k_dev.item())
    steps = 3
    cache = z.QuantCache(L, Hkv, d, layer.q.dtype, DEV, cap_hi=kk + steps, cap_lo=L - kk + 1)
    lens = z.zipvl_quantize_kv(desc, k, v, idx, k_dev, L, cache, status=st)
    torch.cuda.synchronize()
    assert st.item() == 0 and lens.tolist() == [kk, L - kk]
    T = idx[:kk].cpu().numpy()
    ref = oracle.quantize_kv(to_np(layer.k), to_np(layer.v), T, storage)
    _check_blocks(_blocks_from_gpu(cache, kk, L - kk), ref)
    # the cache is several times smaller than the 16-bit one
    assert cache.nbytes(kk, L - kk) < 0.36 * (2 * L * Hkv * d * 2)
    # decode steps with appends, against the oracle on its own copy of the cache
    code = z.ZIPVL_F16 if storage == "f16" else z.ZIPVL_BF16
    ddesc = z.zipvl_decode_desc(1, Hq, Hkv, d, code, 0.0)
    g = torch.Generator().manual_seed(5)
    for s_ in range(steps):
        qn = torch.randn(1, Hq, d, generator=g).to(layer.q.dtype)
        kn = torch.randn(1, Hkv, d, generator=g).to(layer.q.dtype)
        vn = torch.randn(1, Hkv, d, generator=g).to(layer.q.dtype)
        out = z.zipvl_decode_quant(ddesc, qn.to(DEV), kn.to(DEV), vn.to(DEV), cache, L + steps, status=st)
        want = oracle.decode_step_quant(to_np(qn), to_np(kn), to_np(vn), ref, Hkv, storage)
        check_attention(to_np(out), want, layer.q.dtype)
        assert cache.lens.tolist() == [kk + s_ + 1, L - kk]
    assert st.item() == 0
    # the appended rows carry the oracle's codes and parameters too
    _check_blocks(_blocks_from_gpu(cache, kk + steps, L - kk), ref)
    # and the quantised attention stays close to the attention over the 16-bit cache (what the
    # quantisation costs: 4-bit tokens of T, 2-bit others)
    out_q = z.zipvl_decode_quant(ddesc, qn.to(DEV), None, None, cache, L + steps, status=st)
    want_q = oracle.decode_step_quant(to_np(qn), None, None, ref, Hkv, storage)
    check_attention(to_np(out_q), want_q, layer.q.dtype)
    # a full 4-bit block: the append is refused and flagged, the attention still runs
    z.zipvl_decode_quant(ddesc, qn.to(DEV), kn.to(DEV), vn.to(DEV), cache, L + steps, status=st)
    torch.cuda.synchronize()
    assert st.item() & z.DEV_CAPACITY and cache.lens.tolist() == [kk + steps, L - kk]


def test_quantise_reports_small_blocks(zipvl):
    z = zipvl
    layer = W.heavy_key_layer(L_visual=300, L_text=20, H=2, seed=85)
    q, k, v, probe = (t.to(DEV) for t in (layer.q, layer.k, layer.v, layer.probe_pos))
    desc = z.layer_desc(q, k)
    acc, norm = z.zipvl_score(desc, q, k, probe)
    k_dev, idx = z.zipvl_select(acc, norm, layer.tau)
    kk = int(k_dev.item())
    cache = z.QuantCache(layer.L, 2, 128, torch.bfloat16, DEV, cap_hi=kk - 5, cap_lo=layer.L - kk)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    lens = z.zipvl_quantize_kv(desc, k, v, idx, k_dev, layer.L, cache, status=st)
    torch.cuda.synchronize()
    assert st.item() & z.DEV_CAPACITY and lens.tolist() == [kk - 5, layer.L - kk]


@pytest.mark.parametrize("case", ["bf16_mha_d128", "fp16_gqa2_d64"])
def test_batched_decode_over_quantised_caches(zipvl, case):
    """Four requests of different lengths, each with its own mixed-precision cache, decoded in one
    call per step (three steps with appends, one without): every request against the oracle on
    its own copy of that request's cache, and against the single-request call.  A table entry with
    a NULL block is skipped and reported; the other requests are not touched by it."""
    z = zipvl
    if case == "bf16_mha_d128":
        Hq, Hkv, d, dtype, storage = 8, 8, 128, torch.bfloat16, "bf16"
    else:
        Hq, Hkv, d, dtype, storage = 8, 4, 64, torch.float16, "f16"
    code = z.ZIPVL_F16 if storage == "f16" else z.ZIPVL_BF16
    steps, B = 3, 4
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    caches, refs, twins = [], [], []
    for b, (Lv, Lt) in enumerate([(700, 33), (64, 20), (1500, 41), (300, 7)]):
        layer = W.heavy_key_layer(L_visual=Lv, L_text=Lt, H=Hq, Hkv=Hkv, d=d, seed=90 + b, dtype=dtype)
        q, k, v, probe = (t.to(DEV) for t in (layer.q, layer.k, layer.v, layer.probe_pos))
        desc = z.layer_desc(q, k)
        acc, norm = z.zipvl_score(desc, q, k, probe, status=st)
        k_dev, idx = z.zipvl_select(acc, norm, layer.tau, status=st)
        kk = int(k_dev.item())
        for group in (caches, twins):          # twins: the same caches for the single-request calls
            c = z.QuantCache(layer.L, Hkv, d, dtype, DEV, cap_hi=kk + steps, cap_lo=layer.L - kk + 1)
            z.zipvl_quantize_kv(desc, k, v, idx, k_dev, layer.L, c, status=st)
            group.append(c)
        refs.append(oracle.quantize_kv(to_np(layer.k), to_np(layer.v), idx[:kk].cpu().numpy(), storage))
    table = z.quant_cache_table(caches, DEV)
    max_len = max(c.cap_hi + c.cap_lo for c in caches)
    bdesc = z.zipvl_decode_desc(B, Hq, Hkv, d, code, 0.0)
    sdesc = z.zipvl_decode_desc(1, Hq, Hkv, d, code, 0.0)
    g = torch.Generator().manual_seed(17)
    for s_ in range(steps + 1):
        append = s_ < steps
        qn = torch.randn(B, Hq, d, generator=g).to(dtype)
        kn = torch.randn(B, Hkv, d, generator=g).to(dtype) if append else None
        vn = torch.randn(B, Hkv, d, generator=g).to(dtype) if append else None
        out = z.zipvl_decode_quant_batch(bdesc, qn.to(DEV), None if kn is None else kn.to(DEV),
                                         None if vn is None else vn.to(DEV), table, max_len, status=st)
        for b in range(B):
            want = oracle.decode_step_quant(to_np(qn[b:b + 1]), None if kn is None else to_np(kn[b:b + 1]),
                                            None if vn is None else to_np(vn[b:b + 1]), refs[b], Hkv, storage)
            check_attention(to_np(out[b:b + 1]), want, dtype)
            one = z.zipvl_decode_quant(sdesc, qn[b:b + 1].to(DEV), None if kn is None else kn[b:b + 1].to(DEV),
                                       None if vn is None else vn[b:b + 1].to(DEV), twins[b], max_len, status=st)
            check_attention(to_np(out[b:b + 1]), to_np(one).astype(np.float64), dtype)
            assert caches[b].lens.tolist() == twins[b].lens.tolist()
    assert st.item() == 0
    for b in range(B):                          # the appended rows: the same bits as the single-request path
        n_hi, n_lo = caches[b].lens.tolist()
        got, twin = _blocks_from_gpu(caches[b], n_hi, n_lo), _blocks_from_gpu(twins[b], n_hi, n_lo)
        for blk in ("hi", "lo"):
            for part in ("k", "v", "p"):
                assert np.array_equal(got[blk][part], twin[blk][part])
    # a broken table entry: request 1 without its 2-bit keys
    bad = table.clone()
    bad[1, 3] = 0
    before = [c.lens.tolist() for c in caches]
    qn = torch.randn(B, Hq, d, generator=g).to(dtype)
    good = z.zipvl_decode_quant_batch(bdesc, qn.to(DEV), None, None, table, max_len, status=st)
    st2 = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = z.zipvl_decode_quant_batch(bdesc, qn.to(DEV), None, None, bad, max_len, status=st2)
    torch.cuda.synchronize()
    assert st2.item() & z.DEV_BAD_INDEX and st.item() == 0
    assert not out[1].float().abs().sum().item()
    for b in (0, 2, 3):
        assert torch.equal(out[b], good[b])
    assert [c.lens.tolist() for c in caches] == before
