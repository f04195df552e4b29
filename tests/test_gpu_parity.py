"""GPU parity: every C-ABI call against the CPU oracle on the same seeded inputs.

All tests here need a B200 (``-m gpu``) and go through libzipvl.so via the thin
binding; the oracle is only ever the checker."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_08584_b200 import workloads as W
from parity import check_attention, check_scores, check_select, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def layer_cases():
    return {
        "tiny_fp32": lambda: W.tiny_layer(),
        "tiny_fp32_d128": lambda: W.tiny_layer(L=333, H=2, d=128, n_probe=40, seed=11),
        "llava7b_small_bf16": lambda: W.heavy_key_layer(L_visual=1150, L_text=64, H=8, seed=21),
        "bf16_d64": lambda: W.heavy_key_layer(L_visual=500, L_text=41, H=4, d=64, seed=22),
        "video_gqa_small": lambda: W.video_layer(n_frames=10, Hq=14, Hkv=2, seed=23),
        "aligned_sinks": lambda: W.aligned_sink_layer(L=900, H=4, seed=24),
        "one_token": lambda: W.heavy_key_layer(L_visual=0, L_text=1, H=2, seed=25),
        "five_tokens_all_probes": lambda: W.heavy_key_layer(L_visual=3, L_text=2, H=2, seed=26),
        "ragged_129": lambda: W.heavy_key_layer(L_visual=100, L_text=29, H=3, Hkv=1, seed=27),
        "llava7b_small_fp16": lambda: W.heavy_key_layer(L_visual=1150, L_text=64, H=8, seed=31,
                                                        dtype=torch.float16),
        "fp16_d64": lambda: W.heavy_key_layer(L_visual=300, L_text=33, H=4, d=64, seed=32, dtype=torch.float16),
        # head_dim 96 and 64 on the tensor-core kernels (the front of their 128-wide tiles), with
        # grouped heads and several key tiles; head_dim 96 in fp32 on the CUDA-core kernels
        "bf16_d96_gqa": lambda: W.heavy_key_layer(L_visual=1200, L_text=77, H=6, Hkv=2, d=96, seed=41),
        "fp16_d96": lambda: W.heavy_key_layer(L_visual=400, L_text=19, H=3, d=96, seed=42, dtype=torch.float16),
        "bf16_d64_gqa": lambda: W.heavy_key_layer(L_visual=1300, L_text=64, H=8, Hkv=4, d=64, seed=43),
        "fp32_d96": lambda: W.tiny_layer(L=300, H=2, d=96, n_probe=40, seed=44),
        "video_gqa_small_fp16": lambda: W.video_layer(n_frames=7, Hq=14, Hkv=2, seed=33, dtype=torch.float16),
    }


CASES = layer_cases()


def put(layer):
    return (layer.q.to(DEV), layer.k.to(DEV), layer.v.to(DEV), layer.probe_pos.to(DEV))


def status_word():
    return torch.zeros(1, dtype=torch.int32, device=DEV)


def gpu_pipeline(z, layer, tau=None, mode=0, fixed_k=0, out_mode=None):
    """score -> select -> sparse_prefill -> compact_kv on the GPU."""
    tau = layer.tau if tau is None else tau
    out_mode = z.OUT_PADDED if out_mode is None else out_mode
    q, k, v, probe = put(layer)
    desc = z.layer_desc(q, k)
    st = status_word()
    total = torch.zeros(1, dtype=torch.float64, device=DEV)
    acc, norm = z.zipvl_score(desc, q, k, probe, total=total, status=st)
    kept = torch.zeros(1, dtype=torch.float32, device=DEV)
    k_dev, idx = z.zipvl_select(acc, norm, tau, mode=mode, fixed_k=fixed_k, kept_mass=kept, status=st)
    out = z.zipvl_sparse_prefill(desc, q, k, v, idx, k_dev, layer.L, out_mode=out_mode, status=st)
    kc, vc = torch.zeros_like(k), torch.zeros_like(v)
    n = z.zipvl_compact_kv(desc, k, v, idx, k_dev, layer.L, kc, vc, layer.L, status=st)
    torch.cuda.synchronize()
    return dict(acc=acc.cpu().numpy(), norm=norm.cpu().numpy(), total=float(total.item()),
                k=int(k_dev.item()), idx=idx.cpu().numpy(), out=out, kc=kc, vc=vc,
                len=int(n.item()), kept=float(kept.item()), status=int(st.item()))


@pytest.mark.parametrize("name", list(CASES))
def test_score_parity(zipvl, name):
    layer = CASES[name]()
    q, k, v, probe = put(layer)
    desc = zipvl.layer_desc(q, k)
    total = torch.zeros(1, dtype=torch.float64, device=DEV)
    st = status_word()
    acc, norm = zipvl.zipvl_score(desc, q, k, probe, total=total, status=st)
    torch.cuda.synchronize()
    acc_ref, S = oracle.probe_scores(to_np(layer.q), to_np(layer.k), layer.probe_pos.numpy())
    norm_ref, _ = oracle.normalise(acc_ref, layer.probe_pos.numpy(), layer.n_q_heads)
    check_scores(acc.cpu().numpy(), norm.cpu().numpy(), acc_ref, norm_ref, S)
    assert abs(total.item() - S) <= 1e-5 * S
    # the row-softmax identity quoted under Eq. 7
    assert abs(total.item() - len(layer.probe_pos) * layer.n_q_heads) <= 1e-4 * S
    assert st.item() == 0


@pytest.mark.parametrize("name", list(CASES))
def test_select_on_gpu_scores_is_exact(zipvl, name):
    layer = CASES[name]()
    r = gpu_pipeline(zipvl, layer)
    acc64, norm64 = r["acc"].astype(np.float64), r["norm"].astype(np.float64)
    p, T = check_select(r["k"], r["idx"], acc64, norm64, layer.tau)
    assert abs(r["kept"] - acc64[r["idx"][:r["k"]]].sum() / acc64.sum()) < 1e-5
    assert r["status"] == 0


def test_select_end_to_end_vs_pure_oracle(zipvl):
    layer = CASES["tiny_fp32"]()
    r = gpu_pipeline(zipvl, layer)
    acc_ref, S = oracle.probe_scores(to_np(layer.q), to_np(layer.k), layer.probe_pos.numpy())
    norm_ref, _ = oracle.normalise(acc_ref, layer.probe_pos.numpy(), layer.n_q_heads)
    err = np.abs(r["acc"] - acc_ref)[acc_ref > 1e-6 * S] / acc_ref[acc_ref > 1e-6 * S]
    eps = max(1e-6, 4 * float(err.max()))
    check_select(r["k"], r["idx"], acc_ref, norm_ref, layer.tau, eps=eps)


@pytest.mark.parametrize("L,kind", [(1, "rand"), (2, "rand"), (37, "ties"), (1000, "rand"),
                                    (1024, "onehot"), (1025, "uniform"), (5000, "ties"),
                                    (40000, "rand"), (3000, "wide"), (9000, "wide"),
                                    (3000, "dense"), (9000, "dense")])
def test_select_synthetic_scores(zipvl, L, kind):
    g = torch.Generator().manual_seed(L)
    if kind == "rand":
        acc = torch.rand(L, generator=g) ** 4
    elif kind == "ties":
        acc = torch.randint(1, 6, (L,), generator=g).float() * 0.125
    elif kind == "wide":      # a hundred octaves: the level-1 histogram is sparse and wide
        acc = 10.0 ** (-30.0 * torch.rand(L, generator=g))
    elif kind == "dense":     # thousands of distinct values that share 20 key bits
        acc = 1.0 + 1e-4 * torch.rand(L, generator=g)
    elif kind == "onehot":
        acc = torch.full((L,), 1e-5)
        acc[L // 3] = 50.0
    else:
        acc = torch.ones(L)
    nnz = torch.arange(L, 0, -1).float().clamp(max=64)
    norm = acc / nnz
    a, n = acc.to(DEV), norm.to(DEV)
    a64, n64 = acc.double().numpy(), norm.double().numpy()
    for tau in (0.3, 0.9, 0.97, 1.0):
        for mode in (0, zipvl.BUDGET_BY_NORM, zipvl.TOPK_BY_ACC,
                     zipvl.BUDGET_BY_NORM | zipvl.TOPK_BY_ACC):
            k_dev, idx = zipvl.zipvl_select(a, n, tau, mode=mode)
            bm = oracle.METRIC_NORM if mode & zipvl.BUDGET_BY_NORM else oracle.METRIC_ACC
            tm = oracle.METRIC_ACC if mode & zipvl.TOPK_BY_ACC else oracle.METRIC_NORM
            check_select(int(k_dev.item()), idx.cpu().numpy(), a64, n64, tau,
                         budget_metric=bm, topk_metric=tm)
    for fk in (1, L // 2 + 1, L, L + 7):
        k_dev, idx = zipvl.zipvl_select(a, n, 0.5, fixed_k=fk)
        assert k_dev.item() == min(fk, L)
        check_select(int(k_dev.item()), idx.cpu().numpy(), a64, n64, 0.5, fixed_k=fk)
    # the option outside the paper: the last r positions join T
    for r in (1, 5, L // 3 + 1, L + 2):
        for tau, fk in ((0.3, 0), (0.9, 0), (0.5, max(1, L // 4))):
            k_dev, idx = zipvl.zipvl_select(a, n, tau, mode=zipvl.keep_last(r), fixed_k=fk)
            check_select(int(k_dev.item()), idx.cpu().numpy(), a64, n64, tau, fixed_k=fk, keep_last=r)


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("out_mode", ["padded", "compact"])
def test_sparse_prefill_and_compaction_parity(zipvl, name, out_mode):
    layer = CASES[name]()
    mode = zipvl.OUT_PADDED if out_mode == "padded" else zipvl.OUT_COMPACT
    r = gpu_pipeline(zipvl, layer, out_mode=mode)
    T = r["idx"][:r["k"]]
    ref = oracle.sparse_prefill(to_np(layer.q), to_np(layer.k), to_np(layer.v), T)
    out = to_np(r["out"])
    if out_mode == "padded":
        check_attention(out[T], ref, layer.q.dtype)
        U = np.setdiff1d(np.arange(layer.L), T)
        assert np.all(out[U] == 0), "rows of dropped tokens must be zero"
    else:
        check_attention(out[:r["k"]], ref, layer.q.dtype)
    # compaction: bit-exact gather
    bits = torch.int16 if layer.k.element_size() == 2 else torch.int32
    kc = r["kc"].view(bits).cpu().numpy()
    vc = r["vc"].view(bits).cpu().numpy()
    assert r["len"] == r["k"]
    np.testing.assert_array_equal(kc[:r["k"]], oracle.compact_rows(layer.k.view(bits).numpy(), T))
    np.testing.assert_array_equal(vc[:r["k"]], oracle.compact_rows(layer.v.view(bits).numpy(), T))
    assert r["status"] == 0


@pytest.mark.parametrize("name", ["llava7b_small_bf16", "video_gqa_small", "ragged_129", "tiny_fp32",
                                  "one_token"])
@pytest.mark.parametrize("out_mode", ["padded", "compact"])
def test_fused_prefill_and_compaction_equal_the_two_calls(zipvl, name, out_mode):
    """zipvl_sparse_prefill_compact must reproduce zipvl_sparse_prefill and
    zipvl_compact_kv bit for bit (and so inherits their parity with the oracle)."""
    layer = CASES[name]()
    mode = zipvl.OUT_PADDED if out_mode == "padded" else zipvl.OUT_COMPACT
    r = gpu_pipeline(zipvl, layer, out_mode=mode)
    q, k, v, probe = put(layer)
    desc = zipvl.layer_desc(q, k)
    st = status_word()
    acc, norm = zipvl.zipvl_score(desc, q, k, probe, status=st)
    k_dev, idx = zipvl.zipvl_select(acc, norm, layer.tau, status=st)
    kc, vc = torch.zeros_like(k), torch.zeros_like(v)
    out, n = zipvl.zipvl_sparse_prefill_compact(desc, q, k, v, idx, k_dev, layer.L, kc, vc, layer.L,
                                                out_mode=mode, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and int(n.item()) == r["k"]
    rows = layer.L if out_mode == "padded" else r["k"]
    assert torch.equal(out[:rows], r["out"][:rows])
    assert torch.equal(kc, r["kc"]) and torch.equal(vc, r["vc"])
    # the caches against the oracle as well
    bits = torch.int16 if layer.k.element_size() == 2 else torch.int32
    T = r["idx"][:r["k"]]
    np.testing.assert_array_equal(kc.view(bits).cpu().numpy()[:r["k"]],
                                  oracle.compact_rows(layer.k.view(bits).numpy(), T))


@pytest.mark.parametrize("name", ["llava7b_small_bf16", "video_gqa_small", "ragged_129", "llava7b_small_fp16",
                                  "one_token"])
@pytest.mark.parametrize("out_mode", ["padded", "compact"])
def test_single_tile_attention_kernel_gives_the_bits_of_the_default_one(zipvl, name, out_mode, monkeypatch):
    """The library's second tensor-core attention kernel (one 128-row query tile per thread
    block, two blocks per SM; selected by an environment variable) does the same arithmetic in
    the same order as the default one, which the tests above hold against the oracle: outputs,
    compacted caches and lengths must agree bit for bit."""
    layer = CASES[name]()
    q, k, v, probe = put(layer)
    desc = zipvl.layer_desc(q, k)
    acc, norm = zipvl.zipvl_score(desc, q, k, probe)
    k_dev, idx = zipvl.zipvl_select(acc, norm, layer.tau)
    mode = zipvl.OUT_PADDED if out_mode == "padded" else zipvl.OUT_COMPACT
    res = {}
    for kernel in ("pair", "single"):
        monkeypatch.setenv("ZIPVL_PREFILL_KERNEL", kernel)
        st = status_word()
        kc, vc = torch.zeros_like(k), torch.zeros_like(v)
        out = torch.zeros((layer.L, layer.n_q_heads, layer.head_dim), dtype=q.dtype, device=DEV)
        _, n = zipvl.zipvl_sparse_prefill_compact(desc, q, k, v, idx, k_dev, layer.L, kc, vc, layer.L,
                                                  out=out, out_mode=mode, status=st)
        torch.cuda.synchronize()
        assert st.item() == 0
        res[kernel] = (out, kc, vc, int(n.item()))
    a, b = res["pair"], res["single"]
    assert a[3] == b[3] == int(k_dev.item())
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])


@pytest.mark.parametrize("kind", ["bf16_tensor_core", "fp16_gqa", "fp32_cuda_core"])
def test_batched_calls_equal_the_single_sequence_calls(zipvl, kind):
    """Several sequences of one shape through zipvl_score_batch / zipvl_select_batch /
    zipvl_sparse_prefill_batch: per sequence the bits of the single-sequence calls (which the
    tests above hold against the oracle), and sequence 0 once more against the oracle itself."""
    if kind == "bf16_tensor_core":
        layers = [W.heavy_key_layer(L_visual=700, L_text=64, H=4, seed=51 + i, probe_seed=500 + i,
                                    heavy_frac=0.05 + 0.1 * i) for i in range(3)]
    elif kind == "fp16_gqa":
        layers = [W.video_layer(n_frames=5, Hq=14, Hkv=2, seed=61 + i, dtype=torch.float16) for i in range(2)]
    else:
        layers = [W.tiny_layer(L=333, H=2, d=64, n_probe=40, seed=71 + i) for i in range(2)]
    n_seq, L = len(layers), layers[0].L
    q = torch.stack([l.q for l in layers]).to(DEV)
    k = torch.stack([l.k for l in layers]).to(DEV)
    v = torch.stack([l.v for l in layers]).to(DEV)
    probe = torch.stack([l.probe_pos for l in layers]).to(DEV)
    tau = layers[0].tau
    st = status_word()
    acc, norm = zipvl.zipvl_score_batch(q, k, probe, status=st)
    k_dev, idx = zipvl.zipvl_select_batch(acc, norm, tau, status=st)
    Hkv, d = k.shape[2], k.shape[3]
    cap = L + 3
    kc = torch.zeros(n_seq, cap, Hkv, d, dtype=k.dtype, device=DEV)
    vc = torch.zeros_like(kc)
    out, n = zipvl.zipvl_sparse_prefill_batch(q, k, v, idx, k_dev, L, kc, vc, cap, status=st)
    out_c, _ = zipvl.zipvl_sparse_prefill_batch(q, k, v, idx, k_dev, L, out_mode=zipvl.OUT_COMPACT, status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    ks = k_dev.tolist()
    assert len(set(ks)) > 1 or n_seq == 1, "the sequences should keep different numbers of tokens"
    for z in range(n_seq):
        desc = zipvl.layer_desc(q[z], k[z])
        a1, n1 = zipvl.zipvl_score(desc, q[z], k[z], probe[z])
        kd1, idx1 = zipvl.zipvl_select(a1, n1, tau)
        kc1, vc1 = torch.zeros(cap, Hkv, d, dtype=k.dtype, device=DEV), torch.zeros(cap, Hkv, d, dtype=k.dtype, device=DEV)
        o1, len1 = zipvl.zipvl_sparse_prefill_compact(desc, q[z], k[z], v[z], idx1, kd1, L, kc1, vc1, cap)
        oc1 = zipvl.zipvl_sparse_prefill(desc, q[z], k[z], v[z], idx1, kd1, L, out_mode=zipvl.OUT_COMPACT)
        torch.cuda.synchronize()
        assert torch.equal(acc[z], a1) and torch.equal(norm[z], n1)
        assert kd1.item() == ks[z] and torch.equal(idx[z], idx1)
        assert torch.equal(out[z], o1) and n[z].item() == len1.item() == ks[z]
        assert torch.equal(kc[z], kc1) and torch.equal(vc[z], vc1)
        assert torch.equal(out_c[z][:ks[z]], oc1[:ks[z]])
    # sequence 0 against the oracle
    l0 = layers[0]
    qf, kf, vf = to_np(l0.q), to_np(l0.k), to_np(l0.v)
    acc_ref, S = oracle.probe_scores(qf, kf, l0.probe_pos.numpy())
    norm_ref, _ = oracle.normalise(acc_ref, l0.probe_pos.numpy(), l0.n_q_heads)
    check_scores(acc[0].cpu().numpy(), norm[0].cpu().numpy(), acc_ref, norm_ref, S)
    T = idx[0][:ks[0]].cpu().numpy()
    ref = oracle.sparse_prefill(qf, kf, vf, T)
    check_attention(to_np(out[0])[T], ref, l0.q.dtype)


def test_batched_select_of_long_rows(zipvl):
    """Rows longer than one CTA holds go through the multi-CTA kernel sequence by sequence."""
    g = torch.Generator().manual_seed(9)
    acc = (torch.rand(3, 5000, generator=g) ** 3).to(DEV)
    norm = (acc.cpu() * torch.rand(3, 5000, generator=g)).to(DEV)
    k_dev, idx = zipvl.zipvl_select_batch(acc, norm, 0.9)
    torch.cuda.synchronize()
    for z in range(3):
        check_select(int(k_dev[z].item()), idx[z].cpu().numpy(), acc[z].cpu().numpy().astype(np.float64),
                     norm[z].cpu().numpy().astype(np.float64), 0.9)


def test_fused_prefill_compaction_reports_a_small_cache(zipvl):
    layer = CASES["llava7b_small_bf16"]()
    q, k, v, probe = put(layer)
    desc = zipvl.layer_desc(q, k)
    st = status_word()
    acc, norm = zipvl.zipvl_score(desc, q, k, probe, status=st)
    k_dev, idx = zipvl.zipvl_select(acc, norm, layer.tau, status=st)
    cap = 100
    kc = torch.zeros(cap + 4, layer.n_kv_heads, layer.head_dim, dtype=k.dtype, device=DEV)
    vc = torch.zeros_like(kc)
    out, n = zipvl.zipvl_sparse_prefill_compact(desc, q, k, v, idx, k_dev, layer.L, kc, vc, cap, status=st)
    torch.cuda.synchronize()
    assert int(n.item()) == cap and int(st.item()) & zipvl.DEV_CAPACITY
    T = idx[:cap].long()
    assert torch.equal(kc[:cap], k[T]) and torch.equal(vc[:cap], v[T])
    assert torch.count_nonzero(kc[cap:]) == 0            # nothing written past the capacity


def test_tau_one_is_dense_attention(zipvl):
    layer = CASES["llava7b_small_bf16"]()
    r = gpu_pipeline(zipvl, layer, tau=1.0)
    assert r["k"] == layer.L and np.array_equal(r["idx"], np.arange(layer.L))
    rows = np.unique(np.linspace(0, layer.L - 1, 97).astype(np.int32))
    ref = oracle.sparse_prefill(to_np(layer.q), to_np(layer.k), to_np(layer.v),
                                np.arange(layer.L), rows=rows)
    check_attention(to_np(r["out"])[rows], ref, layer.q.dtype)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_running_max_growth_rescales_the_accumulator(zipvl, dtype):
    """Keys that lift the row maximum by more than 2^32 (2^8 for IEEE half) long after the
    first key tile: the lazy running max has to move and the accumulator must be rescaled."""
    layer = W.growing_max_layer(dtype=dtype)
    assert 20.0 * 20.0 * 1.4427 / np.sqrt(128) > 32 + 8
    r = gpu_pipeline(zipvl, layer, tau=1.0)
    assert r["k"] == layer.L
    ref = oracle.sparse_prefill(to_np(layer.q), to_np(layer.k), to_np(layer.v), np.arange(layer.L))
    check_attention(to_np(r["out"]), ref, layer.q.dtype)
    assert r["status"] == 0


@pytest.mark.parametrize("name", ["llava7b_small_bf16", "video_gqa_small", "tiny_fp32", "bf16_d64",
                                  "llava7b_small_fp16"])
def test_token_strided_views_of_a_fused_qkv_buffer(zipvl, name):
    """Q, K, V as slices of one [L, (Hq + 2 Hkv) d] buffer (token strides in the layer
    descriptor): every call must give the bits it gives on contiguous copies."""
    layer = CASES[name]()
    L, Hq, Hkv, d = layer.L, layer.n_q_heads, layer.n_kv_heads, layer.head_dim
    fused = torch.cat([layer.q.reshape(L, -1), layer.k.reshape(L, -1), layer.v.reshape(L, -1)], dim=1).to(DEV)
    qv = fused[:, :Hq * d].unflatten(1, (Hq, d))
    kv = fused[:, Hq * d:(Hq + Hkv) * d].unflatten(1, (Hkv, d))
    vv = fused[:, (Hq + Hkv) * d:].unflatten(1, (Hkv, d))
    assert not qv.is_contiguous() and qv.stride(0) == (Hq + 2 * Hkv) * d
    q, k, v, probe = put(layer)
    res = []
    for (a, b, c) in ((q, k, v), (qv, kv, vv)):
        desc = zipvl.layer_desc(a, b)
        st = status_word()
        acc, norm = zipvl.zipvl_score(desc, a, b, probe, status=st)
        k_dev, idx = zipvl.zipvl_select(acc, norm, layer.tau, status=st)
        out = zipvl.zipvl_sparse_prefill(desc, a, b, c, idx, k_dev, L, status=st)
        kc, vc = torch.zeros_like(k), torch.zeros_like(v)
        zipvl.zipvl_compact_kv(desc, b, c, idx, k_dev, L, kc, vc, L, status=st)
        out2, kc2, vc2 = torch.empty_like(out), torch.zeros_like(k), torch.zeros_like(v)
        zipvl.zipvl_sparse_prefill_compact(desc, a, b, c, idx, k_dev, L, kc2, vc2, L, out=out2, status=st)
        torch.cuda.synchronize()
        assert st.item() == 0
        res.append((acc, norm, idx, out, kc, vc, out2, kc2, vc2))
    for x, y in zip(res[0], res[1]):
        assert torch.equal(x, y)


@pytest.mark.parametrize("name", ["llava7b_small_bf16", "tiny_fp32"])
def test_softmax_scale_override(zipvl, name):
    """A softmax scale other than 1/sqrt(d) in the layer descriptor reaches every step:
    scores, the set they select, attention and decode, each against the oracle at that scale."""
    layer = CASES[name]()
    scale = 0.5 / np.sqrt(layer.head_dim)
    q, k, v, probe = put(layer)
    desc = zipvl.layer_desc(q, k, softmax_scale=scale)
    st = status_word()
    acc, norm = zipvl.zipvl_score(desc, q, k, probe, status=st)
    acc_ref, S = oracle.probe_scores(to_np(layer.q), to_np(layer.k), layer.probe_pos.numpy(), scale=scale)
    norm_ref, _ = oracle.normalise(acc_ref, layer.probe_pos.numpy(), layer.n_q_heads)
    check_scores(acc.cpu().numpy(), norm.cpu().numpy(), acc_ref, norm_ref, S)
    # ... and differ from the default-scale scores (the override is not ignored)
    acc0, _ = zipvl.zipvl_score(zipvl.layer_desc(q, k), q, k, probe)
    assert not torch.allclose(acc, acc0, rtol=1e-3)
    k_dev, idx = zipvl.zipvl_select(acc, norm, layer.tau, status=st)
    out = zipvl.zipvl_sparse_prefill(desc, q, k, v, idx, k_dev, layer.L, out_mode=zipvl.OUT_COMPACT, status=st)
    torch.cuda.synchronize()
    kk = int(k_dev.item())
    T = idx.cpu().numpy()[:kk]
    rows = np.unique(np.linspace(0, kk - 1, 48).astype(np.int64))
    ref = oracle.sparse_prefill(to_np(layer.q), to_np(layer.k), to_np(layer.v), T, scale=scale, rows=rows)
    check_attention(to_np(out)[rows], ref, layer.q.dtype)
    # one decode step over the uncompacted cache at the same scale
    Hq, Hkv, d = layer.n_q_heads, layer.n_kv_heads, layer.head_dim
    code = {torch.bfloat16: zipvl.ZIPVL_BF16, torch.float32: zipvl.ZIPVL_F32}[layer.q.dtype]
    dd = zipvl.zipvl_decode_desc(1, Hq, Hkv, d, code, scale)
    g = torch.Generator().manual_seed(5)
    qn = torch.randn(1, Hq, d, generator=g).to(layer.q.dtype)
    kn, vn = (torch.randn(1, Hkv, d, generator=g).to(layer.q.dtype) for _ in range(2))
    cap = layer.L + 4
    kc = torch.zeros(cap, Hkv, d, dtype=layer.q.dtype)
    vc = torch.zeros_like(kc)
    kc[:layer.L], vc[:layer.L] = layer.k, layer.v
    seq = torch.tensor([layer.L], dtype=torch.int32, device=DEV)
    o = zipvl.zipvl_decode(dd, qn.to(DEV), kn.to(DEV), vn.to(DEV), kc.to(DEV).reshape(-1), vc.to(DEV).reshape(-1),
                           torch.zeros(1, dtype=torch.int64, device=DEV),
                           torch.tensor([cap], dtype=torch.int32, device=DEV), seq, cap, status=st)
    torch.cuda.synchronize()
    kf, vf = kc.float().numpy().reshape(-1).copy(), vc.float().numpy().reshape(-1).copy()
    lens = np.array([layer.L], np.int32)
    ref = oracle.decode_step(to_np(qn), to_np(kn), to_np(vn), kf, vf, np.zeros(1, np.int64), lens, Hkv, scale=scale)
    check_attention(to_np(o), ref, layer.q.dtype)
    assert seq.item() == layer.L + 1 and st.item() == 0


def test_fixed_k_and_metric_modes_through_pipeline(zipvl):
    layer = CASES["aligned_sinks"]()
    r = gpu_pipeline(zipvl, layer, fixed_k=100)
    assert r["k"] == 100
    r = gpu_pipeline(zipvl, layer, mode=zipvl.TOPK_BY_ACC)
    # acc/acc pairing: the kept set itself holds at least tau of the mass
    assert r["kept"] >= layer.tau - 1e-6


def test_two_runs_are_bitwise_identical(zipvl):
    layer = CASES["video_gqa_small"]()
    a, b = gpu_pipeline(zipvl, layer), gpu_pipeline(zipvl, layer)
    assert a["k"] == b["k"] and np.array_equal(a["idx"], b["idx"])
    assert a["acc"].tobytes() == b["acc"].tobytes() and a["norm"].tobytes() == b["norm"].tobytes()
    assert torch.equal(a["out"], b["out"]) and torch.equal(a["kc"], b["kc"])


def test_two_layers_in_flight_on_two_streams(zipvl):
    """The calls keep no hidden state: two different layers run interleaved on two streams
    (each with its own buffers and workspace) give the bits of running each alone."""
    layers = [CASES["llava7b_small_bf16"](), CASES["video_gqa_small"]()]
    alone = [gpu_pipeline(zipvl, lay) for lay in layers]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    bufs = []
    for lay in layers:
        q, k, v, probe = put(lay)
        desc = zipvl.layer_desc(q, k)
        bufs.append(dict(q=q, k=k, v=v, probe=probe, desc=desc, st=status_word(),
                         acc=torch.empty(lay.L, device=DEV), norm=torch.empty(lay.L, device=DEV),
                         k_dev=torch.zeros(1, dtype=torch.int32, device=DEV),
                         idx=torch.empty(lay.L, dtype=torch.int32, device=DEV),
                         out=torch.empty_like(q), kc=torch.zeros_like(k), vc=torch.zeros_like(v),
                         n=torch.zeros(1, dtype=torch.int32, device=DEV),
                         ws=[zipvl.workspace(zipvl.zipvl_workspace_bytes(op, desc, probe.numel()), DEV)
                             for op in (zipvl.OP_SCORE, zipvl.OP_SELECT, zipvl.OP_SPARSE_PREFILL)]))
    torch.cuda.synchronize()
    for it in range(20):
        for lay, b, s in zip(layers, bufs, streams):
            zipvl.zipvl_score(b["desc"], b["q"], b["k"], b["probe"], acc=b["acc"], norm=b["norm"], ws=b["ws"][0],
                              status=b["st"], stream=s)
        for lay, b, s in zip(layers, bufs, streams):
            zipvl.zipvl_select(b["acc"], b["norm"], lay.tau, k_out=b["k_dev"], idx=b["idx"], ws=b["ws"][1],
                               status=b["st"], stream=s)
        for lay, b, s in zip(layers, bufs, streams):
            zipvl.zipvl_sparse_prefill_compact(b["desc"], b["q"], b["k"], b["v"], b["idx"], b["k_dev"], lay.L,
                                               b["kc"], b["vc"], lay.L, out=b["out"], len_out=b["n"],
                                               ws=b["ws"][2], status=b["st"], stream=s)
    torch.cuda.synchronize()
    for b, ref in zip(bufs, alone):
        assert b["st"].item() == 0 and b["k_dev"].item() == ref["k"] == b["n"].item()
        assert np.array_equal(b["idx"].cpu().numpy(), ref["idx"])
        assert torch.equal(b["out"], ref["out"])
        kk = ref["k"]
        assert torch.equal(b["kc"][:kk], ref["kc"][:kk]) and torch.equal(b["vc"][:kk], ref["vc"][:kk])


def test_bad_index_is_reported_not_fatal(zipvl):
    layer = CASES["ragged_129"]()
    q, k, v, probe = put(layer)
    desc = zipvl.layer_desc(q, k)
    idx = torch.arange(layer.L, dtype=torch.int32, device=DEV)
    idx[7] = layer.L + 1000
    k_dev = torch.tensor([layer.L], dtype=torch.int32, device=DEV)
    st = status_word()
    zipvl.zipvl_sparse_prefill(desc, q, k, v, idx, k_dev, layer.L, status=st)
    kc, vc = torch.zeros_like(k), torch.zeros_like(v)
    zipvl.zipvl_compact_kv(desc, k, v, idx, k_dev, layer.L, kc, vc, layer.L, status=st)
    torch.cuda.synchronize()
    assert st.item() & zipvl.DEV_BAD_INDEX
    # k larger than the host bound is clamped and flagged
    st.zero_()
    k_dev.fill_(layer.L)
    n = zipvl.zipvl_compact_kv(desc, k, v, idx.clamp(max=layer.L - 1), k_dev, 50, kc, vc, 50, status=st)
    torch.cuda.synchronize()
    assert n.item() == 50 and st.item() & zipvl.DEV_CAPACITY


@pytest.mark.parametrize("name", ["ragged_129", "tiny_fp32_d128"])     # tensor-core and CUDA-core kernels
def test_negative_index_is_skipped_and_writes_nothing_out_of_bounds(zipvl, name):
    """A negative entry inside [0, k): reported, its row skipped, no store in front of `out`
    (canary rows on both sides stay untouched) and every other row as in the clean run."""
    layer = CASES[name]()
    q, k, v, probe = put(layer)
    L, Hq, d = layer.L, layer.n_q_heads, layer.head_dim
    desc = zipvl.layer_desc(q, k)
    idx = torch.arange(L, dtype=torch.int32, device=DEV)
    k_dev = torch.tensor([L], dtype=torch.int32, device=DEV)
    st = status_word()
    clean = zipvl.zipvl_sparse_prefill(desc, q, k, v, idx, k_dev, L, status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    canary = 77.0
    guard = 16                                          # rows in front of and behind the output
    buf = torch.full((L + 2 * guard, Hq, d), canary, dtype=q.dtype, device=DEV)
    out = buf[guard:guard + L]
    bad = idx.clone()
    bad[3] = -7
    zipvl.zipvl_sparse_prefill(desc, q, k, v, bad, k_dev, L, out=out, status=st)
    torch.cuda.synchronize()
    assert st.item() & zipvl.DEV_BAD_INDEX
    assert torch.all(buf[:guard] == canary) and torch.all(buf[guard + L:] == canary)
    # rows 0..2 do not see entry 3 at all: the bits of the clean run.  The bad entry's own
    # row is not written; the later rows saw an all-zero key and value in its place (the
    # documented stand-in), so they are finite and close to, not equal to, the clean run.
    assert torch.equal(out[:3], clean[:3])
    assert torch.all(out[3] == canary)
    assert torch.isfinite(out[4:].float()).all()
    # the fused call and the compaction see the same list
    st.zero_()
    kc, vc = torch.zeros_like(k), torch.zeros_like(v)
    buf.fill_(canary)
    zipvl.zipvl_sparse_prefill_compact(desc, q, k, v, bad, k_dev, L, kc, vc, L, out=out, status=st)
    torch.cuda.synchronize()
    assert st.item() & zipvl.DEV_BAD_INDEX
    assert torch.all(buf[:guard] == canary) and torch.all(buf[guard + L:] == canary)
    assert torch.equal(kc[4:], k[4:]) and torch.equal(kc[:3], k[:3])


@pytest.mark.parametrize("name", ["ragged_129", "tiny_fp32_d128"])
def test_empty_selection_zeroes_the_output_and_the_cache_length(zipvl, name):
    """k = 0 on the device: the padded output is all zeros, the cache length is 0, for the
    separate calls and for the fused one alike."""
    layer = CASES[name]()
    q, k, v, probe = put(layer)
    L = layer.L
    desc = zipvl.layer_desc(q, k)
    idx = torch.full((L,), -1, dtype=torch.int32, device=DEV)
    k_dev = torch.zeros(1, dtype=torch.int32, device=DEV)
    st = status_word()
    out = torch.full_like(q, 5.0)
    zipvl.zipvl_sparse_prefill(desc, q, k, v, idx, k_dev, L, out=out, status=st)
    kc, vc = torch.zeros_like(k), torch.zeros_like(v)
    n = zipvl.zipvl_compact_kv(desc, k, v, idx, k_dev, L, kc, vc, L, status=st)
    out2 = torch.full_like(q, 5.0)
    n2 = torch.full((1,), 99, dtype=torch.int32, device=DEV)
    zipvl.zipvl_sparse_prefill_compact(desc, q, k, v, idx, k_dev, L, kc, vc, L, out=out2, len_out=n2, status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert not out.any() and not out2.any()
    assert n.item() == 0 and n2.item() == 0


def test_a_nan_key_row_reaches_the_scores_and_is_reported_by_the_selection(zipvl):
    """A NaN in one key row: the tensor-core score kernel (whose heads add their column sums into
    fixed-point totals with integer atomics) still hands out NaN for that key's scores, and the
    selection reports the bad value."""
    layer = W.heavy_key_layer(L_visual=700, L_text=64, H=4, seed=33)
    q, k, probe = layer.q.to(DEV), layer.k.clone(), layer.probe_pos.to(DEV)
    k[300, 1, 5] = float("nan")
    k = k.to(DEV)
    desc = zipvl.layer_desc(q, k)
    st = status_word()
    acc, norm = zipvl.zipvl_score(desc, q, k, probe, status=st)
    torch.cuda.synchronize()
    assert torch.isnan(acc[300]).item() and torch.isnan(norm[300]).item()
    st.zero_()
    zipvl.zipvl_select(acc, norm, 0.9, status=st)
    torch.cuda.synchronize()
    assert st.item() & zipvl.DEV_BAD_VALUE


def test_select_reports_negative_and_nan_scores(zipvl):
    g = torch.Generator().manual_seed(3)
    acc = torch.rand(500, generator=g).to(DEV)
    norm = torch.rand(500, generator=g).to(DEV)
    st = status_word()
    zipvl.zipvl_select(acc, norm, 0.9, status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    for bad_val, which in ((-1.0, 0), (float("nan"), 1)):
        a, n = acc.clone(), norm.clone()
        (a if which == 0 else n)[17] = bad_val
        st.zero_()
        k_dev, idx = zipvl.zipvl_select(a, n, 0.9, status=st)
        torch.cuda.synchronize()
        assert st.item() & zipvl.DEV_BAD_VALUE
        kk = int(k_dev.item())
        assert 1 <= kk <= 500 and idx[:kk].min().item() >= 0       # the call still completes


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_survives(zipvl):
    """The wait every tensor-core kernel uses, on a barrier nobody arrives at, with a poll
    limit of a few thousand: the kernel returns, ZIPVL_DEV_TIMEOUT is set, the warp whose
    barrier did complete is unaffected, and the next parity call runs as usual."""
    st = status_word()
    progress = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    zipvl.zipvl_selftest_wait_timeout(4000, progress, st)
    torch.cuda.synchronize()
    assert st.item() == zipvl.DEV_TIMEOUT
    assert progress.tolist() == [1, 0, 0, 0]
    layer = CASES["ragged_129"]()
    r = gpu_pipeline(zipvl, layer)
    assert r["status"] == 0 and r["k"] >= 1


@pytest.mark.parametrize("kernel", ["simt", "tc", "tcp"])
def test_decode_skips_requests_with_impossible_lengths_or_offsets(zipvl, monkeypatch, kernel):
    """seq_lens < 0, seq_lens > capacity and a cache offset off the 16-byte grid: the request
    is skipped (zero output, cache and length untouched) and reported; the other requests of
    the batch are served as usual.  All buffers are in range, so nothing can fault."""
    monkeypatch.setenv("ZIPVL_DECODE_KERNEL", kernel)      # the CUDA-core kernel and both tensor-core ones
    lens, Hq, Hkv, d = [40, 300, 77, 130], 4, 2, 128
    B = len(lens)
    kc, vc, off, cap = build_caches(lens, Hkv, d, torch.bfloat16, 4, seed=8)
    g = torch.Generator().manual_seed(9)
    q = torch.randn(B, Hq, d, generator=g).bfloat16()
    kn = torch.randn(B, Hkv, d, generator=g).bfloat16()
    vn = torch.randn(B, Hkv, d, generator=g).bfloat16()
    desc = zipvl.zipvl_decode_desc(B, Hq, Hkv, d, zipvl.ZIPVL_BF16, 0.0)
    seq_bad = torch.tensor([-3, 300, 77 + 50, 130], dtype=torch.int32)     # request 0 and 2 impossible
    off_bad = off.clone()
    off_bad[3] += 4                                                         # request 3: 8 bytes off
    kc_d, vc_d = kc.to(DEV), vc.to(DEV)
    seq_d = seq_bad.to(DEV)
    st = status_word()
    out = zipvl.zipvl_decode(desc, q.to(DEV), kn.to(DEV), vn.to(DEV), kc_d, vc_d, off_bad.to(DEV),
                             cap.to(DEV), seq_d, max(lens) + 4, status=st)
    torch.cuda.synchronize()
    assert st.item() & zipvl.DEV_BAD_INDEX
    assert seq_d.tolist() == [-3, 301, 127, 130]
    assert not out[0].any() and not out[2].any() and not out[3].any()
    # request 1 is the oracle's answer
    ko, vo = to_np(kc).copy(), to_np(vc).copy()
    seqo = np.array(lens, np.int32)
    ref = oracle.decode_step(to_np(q), to_np(kn), to_np(vn), ko, vo, off.numpy(), seqo, Hkv)
    check_attention(to_np(out)[1], ref[1], torch.bfloat16)
    # and only request 1's cache row changed
    kc_after = kc_d.cpu()
    row = Hkv * d
    o1 = int(off[1]) + 300 * row
    assert torch.equal(kc_after[o1:o1 + row], kn[1].reshape(-1))
    kc_after[o1:o1 + row] = kc[o1:o1 + row]
    assert torch.equal(kc_after, kc)


def test_all_rows_as_probes_on_16_bit_inputs(zipvl):
    """More probe rows than one tensor-core tile holds (the "all tokens" probe strategy of the
    supplementary ablation at L = 300): exact full-attention column sums on bf16 inputs."""
    layer = W.heavy_key_layer(L_visual=260, L_text=40, H=4, seed=41)
    layer.probe_pos = torch.arange(layer.L, dtype=torch.int32)
    r = gpu_pipeline(zipvl, layer)
    assert r["status"] == 0
    qf, kf = to_np(layer.q), to_np(layer.k)
    acc_ref, S = oracle.probe_scores(qf, kf, layer.probe_pos.numpy())
    norm_ref, nnz = oracle.normalise(acc_ref, layer.probe_pos.numpy(), layer.n_q_heads)
    assert np.array_equal(nnz, layer.L - np.arange(layer.L))
    check_scores(r["acc"], r["norm"], acc_ref, norm_ref, S)
    check_select(r["k"], r["idx"], r["acc"].astype(np.float64), r["norm"].astype(np.float64), layer.tau)


def _tiny_shape_case(zipvl, L, H, G, d, n_probe, tau, dtype, seed):
    Hkv = H
    Hq = H * G
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(L, Hq, d, generator=g).to(dtype)
    k = (torch.randn(L, Hkv, d, generator=g) * (1.0 + 2.0 * (torch.rand(L, 1, 1, generator=g) < 0.2))).to(dtype)
    v = torch.randn(L, Hkv, d, generator=g).to(dtype)
    P = min(n_probe, L)
    # P distinct rows, ascending, the last row always among them
    probe = torch.unique(torch.cat([torch.randperm(L, generator=g)[:P - 1],
                                    torch.tensor([L - 1])])).to(torch.int32)
    layer = W.Layer("tiny_shape", q, k, v, probe, tau)
    r = gpu_pipeline(zipvl, layer)
    assert r["status"] == 0
    qf, kf, vf = to_np(q), to_np(k), to_np(v)
    acc_ref, S = oracle.probe_scores(qf, kf, probe.numpy())
    norm_ref, _ = oracle.normalise(acc_ref, probe.numpy(), Hq)
    err = check_scores(r["acc"], r["norm"], acc_ref, norm_ref, S)
    check_select(r["k"], r["idx"], r["acc"].astype(np.float64), r["norm"].astype(np.float64), tau)
    check_select(r["k"], r["idx"], acc_ref, norm_ref, tau, eps=max(1e-6, 4 * err))
    T = r["idx"][: r["k"]]
    ref = oracle.sparse_prefill(qf, kf, vf, T)
    out = to_np(r["out"])
    check_attention(out[T], ref, dtype)
    assert not out[np.setdiff1d(np.arange(L), T)].any()
    Tl = torch.from_numpy(T.astype(np.int64))
    assert r["len"] == r["k"] and torch.equal(r["kc"][: r["k"]].cpu(), k[Tl]) and torch.equal(r["vc"][: r["k"]].cpu(), v[Tl])


def test_generated_tiny_shapes(zipvl):
    """Property-style sweep over small shapes drawn by hypothesis (fixed seed): odd lengths,
    one token, more probes than tokens, one probe, grouped heads, every storage type, budgets
    from one token to everything -- the whole chain against the oracle."""
    from hypothesis import HealthCheck, given, seed, settings
    from hypothesis import strategies as hs

    @seed(20241008)
    @settings(max_examples=40, deadline=None, derandomize=True,
              suppress_health_check=list(HealthCheck))
    @given(L=hs.integers(1, 300), H=hs.integers(1, 3), G=hs.sampled_from([1, 2, 7]),
           d=hs.sampled_from([64, 128]), n_probe=hs.sampled_from([1, 5, 64, 128, 400]),
           tau=hs.sampled_from([0.3, 0.9, 0.97, 1.0]),
           dtype=hs.sampled_from([torch.bfloat16, torch.float16, torch.float32]),
           s=hs.integers(0, 10 ** 6))
    def run(L, H, G, d, n_probe, tau, dtype, s):
        _tiny_shape_case(zipvl, L, H, G, d, n_probe, tau, dtype, s)

    run()


# ----------------------------------------------------------------------------
# decode (Algorithm 2)
# ----------------------------------------------------------------------------
def build_caches(lens, Hkv, d, dtype, extra, seed):
    g = torch.Generator().manual_seed(seed)
    cap = [n + extra for n in lens]
    off = np.concatenate([[0], np.cumsum([c * Hkv * d for c in cap[:-1]])]).astype(np.int64)
    total = int(sum(c * Hkv * d for c in cap))
    kc = torch.zeros(total, dtype=dtype)
    vc = torch.zeros(total, dtype=dtype)
    for b, n in enumerate(lens):
        kc[off[b]: off[b] + n * Hkv * d] = torch.randn(n * Hkv * d, generator=g).to(dtype)
        vc[off[b]: off[b] + n * Hkv * d] = torch.randn(n * Hkv * d, generator=g).to(dtype)
    return kc, vc, torch.from_numpy(off), torch.tensor(cap, dtype=torch.int32)


@pytest.mark.parametrize("lens,Hq,Hkv,d,dtype", [
    ([700, 1, 300, 1025, 17], 8, 8, 128, torch.bfloat16),
    ([513, 40, 2000], 14, 2, 128, torch.bfloat16),
    ([100, 259], 4, 1, 64, torch.bfloat16),
    ([600, 33, 1300], 8, 2, 128, torch.float16),
    ([90, 257], 4, 4, 64, torch.float16),
    ([300, 7], 4, 4, 64, torch.float32),
    ([129], 6, 2, 128, torch.float32),
    ([400, 130, 1], 6, 2, 96, torch.bfloat16),
    ([900, 259, 3], 14, 2, 64, torch.bfloat16),
    ([257, 90], 4, 4, 96, torch.float16),
    ([300, 7], 4, 2, 96, torch.float32),
    # grouped-query heads on the tensor cores: 2, 7, 16 and 32 query heads per kv head, an empty
    # request, lengths of one row, a ragged last tile, more than one chunk per request
    ([300, 1000], 4, 2, 128, torch.bfloat16),
    ([5000, 129, 0, 3000, 1], 28, 4, 128, torch.bfloat16),
    ([2100, 640], 32, 2, 128, torch.float16),
    ([1500, 127], 32, 1, 128, torch.bfloat16),
])
def test_decode_parity(zipvl, lens, Hq, Hkv, d, dtype):
    B, steps = len(lens), 3
    kc, vc, off, cap = build_caches(lens, Hkv, d, dtype, steps, seed=sum(lens))
    g = torch.Generator().manual_seed(99)
    code = {torch.bfloat16: zipvl.ZIPVL_BF16, torch.float32: zipvl.ZIPVL_F32, torch.float16: zipvl.ZIPVL_F16}[dtype]
    desc = zipvl.zipvl_decode_desc(B, Hq, Hkv, d, code, 0.0)
    kc_d, vc_d, off_d, cap_d = kc.to(DEV), vc.to(DEV), off.to(DEV), cap.to(DEV)
    seq_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    kc_o, vc_o = kc.float().numpy().copy(), vc.float().numpy().copy()
    seq_o = np.array(lens, np.int32)
    st = status_word()
    max_len = max(lens) + steps
    for step in range(steps):
        q = torch.randn(B, Hq, d, generator=g).to(dtype)
        kn = torch.randn(B, Hkv, d, generator=g).to(dtype)
        vn = torch.randn(B, Hkv, d, generator=g).to(dtype)
        out = zipvl.zipvl_decode(desc, q.to(DEV), kn.to(DEV), vn.to(DEV), kc_d, vc_d, off_d, cap_d,
                                 seq_d, max_len, status=st)
        ref = oracle.decode_step(to_np(q), to_np(kn), to_np(vn), kc_o, vc_o, off.numpy(), seq_o, Hkv)
        check_attention(to_np(out), ref, dtype)
        assert np.array_equal(seq_d.cpu().numpy(), seq_o)
    # caches after the appends are identical (appended rows are copied bit for bit)
    assert np.array_equal(kc_d.float().cpu().numpy(), kc_o)
    assert np.array_equal(vc_d.float().cpu().numpy(), vc_o)
    # no new token: nothing is appended, lengths stay
    out2 = zipvl.zipvl_decode(desc, q.to(DEV), None, None, kc_d, vc_d, off_d, cap_d, seq_d,
                              max_len, status=st)
    ref2 = oracle.decode_step(to_np(q), None, None, kc_o, vc_o, off.numpy(), seq_o, Hkv)
    check_attention(to_np(out2), ref2, dtype)
    assert st.item() == 0
    # full cache: the append is refused and flagged, attention still runs
    zipvl.zipvl_decode(desc, q.to(DEV), kn.to(DEV), vn.to(DEV), kc_d, vc_d, off_d, cap_d, seq_d,
                       max_len, status=st)
    torch.cuda.synchronize()
    assert st.item() & zipvl.DEV_CAPACITY and np.array_equal(seq_d.cpu().numpy(), seq_o)


@pytest.mark.parametrize("lens,Hq,Hkv,d,dtype", [
    ([513, 40, 2000], 14, 2, 128, torch.bfloat16),
    ([5000, 129, 0, 3000, 1], 28, 4, 128, torch.bfloat16),
    ([2100, 640], 32, 2, 128, torch.float16),
    ([900, 259, 3], 14, 2, 64, torch.bfloat16),          # narrower heads: the front of the 128-wide tiles
    ([400, 1300], 12, 4, 96, torch.float16),
])
def test_decode_parity_on_the_persistent_kernel(zipvl, monkeypatch, lens, Hq, Hkv, d, dtype):
    """The decode parity test (three steps with appends, a step without, a full cache) with the
    persistent tensor-core kernel forced: by default it only takes large batches."""
    monkeypatch.setenv("ZIPVL_DECODE_KERNEL", "tcp")
    test_decode_parity(zipvl, lens, Hq, Hkv, d, dtype)


@pytest.mark.parametrize("lens,Hq,Hkv,dtype,page_rows", [
    ([513, 40, 2000, 0], 16, 4, torch.bfloat16, 16),
    ([3000, 100], 28, 4, torch.float16, 256),
])
def test_paged_decode_parity_on_the_persistent_kernel(zipvl, monkeypatch, lens, Hq, Hkv, dtype, page_rows):
    monkeypatch.setenv("ZIPVL_DECODE_KERNEL", "tcp")
    test_paged_decode_parity(zipvl, lens, Hq, Hkv, 128, dtype, page_rows)


@pytest.mark.parametrize("kernel,lens,Hq,Hkv", [
    ("tc", [700, 130, 2600], 8, 4),        # two query heads per kv head: the CUDA-core kernel by default
    ("simt", [700, 130, 2600], 14, 2),     # seven: the tensor-core kernel by default
    ("tc", [4000], 64, 2),                 # thirty-two, several tiles per CTA
    ("tcp", [700, 130, 2600], 14, 2),      # the persistent kernel (large batches by default)
    ("tcp", [4000, 129], 64, 2),           # thirty-two heads: one set of query rows
    ("tcp", [30000, 9000, 128, 0, 5000], 28, 4),   # long runs of tiles per CTA, an empty request
])
def test_decode_kernel_choice_can_be_forced_and_both_match_the_oracle(zipvl, monkeypatch, kernel, lens, Hq, Hkv):
    """ZIPVL_DECODE_KERNEL picks the grouped-query decode kernel; either choice has to match the
    oracle, repeat bit for bit, and agree with the other one within the attention tolerance."""
    d, dtype, B = 128, torch.bfloat16, len(lens)
    kc, vc, off, cap = build_caches(lens, Hkv, d, dtype, 2, seed=7 * sum(lens))
    g = torch.Generator().manual_seed(5)
    q = torch.randn(B, Hq, d, generator=g).to(dtype)
    desc = zipvl.zipvl_decode_desc(B, Hq, Hkv, d, zipvl.ZIPVL_BF16, 0.0)
    kc_d, vc_d, off_d, cap_d = kc.to(DEV), vc.to(DEV), off.to(DEV), cap.to(DEV)
    seq_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    ref = oracle.decode_step(to_np(q), None, None, kc.float().numpy(), vc.float().numpy(), off.numpy(),
                             np.array(lens, np.int32), Hkv)
    outs = {}
    for which in (kernel, "simt" if kernel != "simt" else "tc"):
        if Hq // Hkv > 8 and which == "simt":
            continue                        # more than eight query heads per kv head: tensor cores only
        monkeypatch.setenv("ZIPVL_DECODE_KERNEL", which)
        st = status_word()
        a = zipvl.zipvl_decode(desc, q.to(DEV), None, None, kc_d, vc_d, off_d, cap_d, seq_d, max(lens), status=st)
        b = zipvl.zipvl_decode(desc, q.to(DEV), None, None, kc_d, vc_d, off_d, cap_d, seq_d, max(lens), status=st)
        assert st.item() == 0 and torch.equal(a, b)
        check_attention(to_np(a), ref, dtype)
        outs[which] = a
    if len(outs) == 2:
        a, b = list(outs.values())
        check_attention(to_np(a), to_np(b).astype(np.float64), dtype)


@pytest.mark.parametrize("kernel,B,Hq,Hkv", [
    ("tcp", 700, 8, 2),        # more requests than the CTA has threads: the length scan takes several each
    ("tcp", 1500, 12, 4),      # far more (request, kv head) pairs than CTAs: dozens of segments per CTA
    ("tc", 700, 8, 2),
    ("simt", 700, 8, 8),
    # batch sizes at which the merge kernel runs with four and with two lanes per head (eight in
    # the small batches of the other tests, one in the large ones above)
    ("tcp", 40, 28, 4),
    ("tc", 80, 28, 4),
    ("simt", 40, 32, 32),
])
def test_decode_on_many_short_requests(zipvl, monkeypatch, kernel, B, Hq, Hkv):
    """Hundreds of requests of zero to a few hundred rows, a few long ones among them, one step with
    an appended token: every request's output, length and appended row against the oracle."""
    monkeypatch.setenv("ZIPVL_DECODE_KERNEL", kernel)
    d, dtype = 128, torch.bfloat16
    rng = np.random.default_rng(B + Hq)
    lens = [int(x) for x in rng.integers(0, 400, size=B)]
    for b in rng.choice(B, size=5, replace=False):
        lens[int(b)] = int(rng.integers(2000, 5000))
    lens[3], lens[B - 1] = 0, 1
    kc, vc, off, cap = build_caches(lens, Hkv, d, dtype, 1, seed=B)
    g = torch.Generator().manual_seed(B)
    q = torch.randn(B, Hq, d, generator=g).to(dtype)
    kn = torch.randn(B, Hkv, d, generator=g).to(dtype)
    vn = torch.randn(B, Hkv, d, generator=g).to(dtype)
    desc = zipvl.zipvl_decode_desc(B, Hq, Hkv, d, zipvl.ZIPVL_BF16, 0.0)
    kc_d, vc_d, off_d, cap_d = kc.to(DEV), vc.to(DEV), off.to(DEV), cap.to(DEV)
    seq_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    st = status_word()
    out = zipvl.zipvl_decode(desc, q.to(DEV), kn.to(DEV), vn.to(DEV), kc_d, vc_d, off_d, cap_d, seq_d,
                             max(lens) + 1, status=st)
    ko, vo, seqo = kc.float().numpy().copy(), vc.float().numpy().copy(), np.array(lens, np.int32)
    ref = oracle.decode_step(to_np(q), to_np(kn), to_np(vn), ko, vo, off.numpy(), seqo, Hkv)
    assert st.item() == 0
    check_attention(to_np(out), ref, dtype)
    assert np.array_equal(seq_d.cpu().numpy(), seqo) and np.array_equal(seqo, np.array(lens) + 1)
    assert np.array_equal(kc_d.float().cpu().numpy(), ko) and np.array_equal(vc_d.float().cpu().numpy(), vo)


@pytest.mark.parametrize("lens,Hq,Hkv,d,dtype,page_rows", [
    ([700, 1, 300, 1025, 17, 0], 8, 8, 128, torch.bfloat16, 64),
    ([513, 40, 2000], 14, 2, 128, torch.bfloat16, 128),
    ([100, 259, 64], 4, 1, 64, torch.float16, 16),
    ([300, 7], 4, 4, 64, torch.float32, 64),
    ([300, 70], 6, 2, 96, torch.bfloat16, 32),
    ([513, 40, 2000, 0], 16, 4, 128, torch.bfloat16, 16),
    ([3000, 100], 28, 4, 128, torch.float16, 256),
])
def test_paged_decode_parity(zipvl, lens, Hq, Hkv, d, dtype, page_rows):
    """Decode over caches scattered in pages of a shared pool (shuffled page numbers), three
    steps with appends that cross page boundaries, against the oracle's paged decode."""
    B, steps = len(lens), 3
    g = torch.Generator().manual_seed(sum(lens) + page_rows)
    pages_per = [-(-(n + steps) // page_rows) for n in lens]
    max_pages = max(pages_per)
    n_pages = sum(pages_per) + 3
    perm = torch.randperm(n_pages, generator=g)
    table = torch.full((B, max_pages), -1, dtype=torch.int32)
    pos = 0
    for b in range(B):
        table[b, :pages_per[b]] = perm[pos:pos + pages_per[b]].to(torch.int32)
        pos += pages_per[b]
    k_pages = torch.randn(n_pages, page_rows, Hkv, d, generator=g).to(dtype)
    v_pages = torch.randn(n_pages, page_rows, Hkv, d, generator=g).to(dtype)
    cap = torch.tensor([p_ * page_rows for p_ in pages_per], dtype=torch.int32)
    code = {torch.bfloat16: zipvl.ZIPVL_BF16, torch.float32: zipvl.ZIPVL_F32, torch.float16: zipvl.ZIPVL_F16}[dtype]
    desc = zipvl.zipvl_decode_desc(B, Hq, Hkv, d, code, 0.0)
    kp_d, vp_d, table_d, cap_d = k_pages.to(DEV), v_pages.to(DEV), table.to(DEV), cap.to(DEV)
    seq_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
    kp_o, vp_o = k_pages.float().numpy().copy(), v_pages.float().numpy().copy()
    table_o = table.clamp(min=0).numpy()            # the oracle never touches the unused entries
    seq_o = np.array(lens, np.int32)
    st = status_word()
    max_len = max(lens) + steps
    for step in range(steps):
        q = torch.randn(B, Hq, d, generator=g).to(dtype)
        kn = torch.randn(B, Hkv, d, generator=g).to(dtype)
        vn = torch.randn(B, Hkv, d, generator=g).to(dtype)
        out = zipvl.zipvl_decode_paged(desc, q.to(DEV), kn.to(DEV), vn.to(DEV), kp_d, vp_d, table_d, cap_d,
                                       seq_d, max_len, status=st)
        ref = oracle.decode_step_paged(to_np(q), to_np(kn), to_np(vn), kp_o, vp_o, table_o, seq_o)
        check_attention(to_np(out), ref, dtype)
        assert np.array_equal(seq_d.cpu().numpy(), seq_o)
    assert st.item() == 0
    # the pools after the appends are identical (appended rows are copied bit for bit)
    assert np.array_equal(kp_d.float().cpu().numpy(), kp_o) and np.array_equal(vp_d.float().cpu().numpy(), vp_o)
    # a page number outside the pool: reported, the rows of that page left out, nothing faults
    bad = table_d.clone()
    bad[0, 0] = n_pages + 5
    zipvl.zipvl_decode_paged(desc, q.to(DEV), None, None, kp_d, vp_d, bad, cap_d, seq_d, max_len, status=st)
    torch.cuda.synchronize()
    assert st.item() & zipvl.DEV_BAD_INDEX


def test_decode_on_compacted_cache_matches_oracle_pipeline(zipvl):
    """prefill -> compaction -> decode chained on the device without host sync of k."""
    layer = CASES["llava7b_small_bf16"]()
    r = gpu_pipeline(zipvl, layer)
    Hq, Hkv, d = layer.n_q_heads, layer.n_kv_heads, layer.head_dim
    desc = zipvl.zipvl_decode_desc(1, Hq, Hkv, d, 0, 0.0)
    g = torch.Generator().manual_seed(5)
    q = torch.randn(1, Hq, d, generator=g).bfloat16()
    kn = torch.randn(1, Hkv, d, generator=g).bfloat16()
    vn = torch.randn(1, Hkv, d, generator=g).bfloat16()
    cap = layer.L + 8
    kc = torch.zeros(cap, Hkv, d, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    kc[:layer.L], vc[:layer.L] = r["kc"], r["vc"]
    seq = torch.tensor([r["len"]], dtype=torch.int32, device=DEV)
    out = zipvl.zipvl_decode(desc, q.to(DEV), kn.to(DEV), vn.to(DEV), kc, vc,
                             torch.zeros(1, dtype=torch.int64, device=DEV),
                             torch.tensor([cap], dtype=torch.int32, device=DEV), seq, cap)
    T = r["idx"][:r["k"]]
    kco = np.zeros(cap * Hkv * d, np.float32)
    vco = np.zeros_like(kco)
    kco[: len(T) * Hkv * d] = to_np(layer.k)[T].ravel()
    vco[: len(T) * Hkv * d] = to_np(layer.v)[T].ravel()
    seqo = np.array([len(T)], np.int32)
    ref = oracle.decode_step(to_np(q), to_np(kn), to_np(vn), kco, vco, np.zeros(1, np.int64), seqo, Hkv)
    check_attention(to_np(out), ref, torch.bfloat16)
    assert seq.item() == len(T) + 1


def test_prefill_layer_host_entry_point(zipvl):
    layer = CASES["ragged_129"]()
    desc = zipvl.zipvl_layer(layer.L, layer.n_q_heads, layer.n_kv_heads, layer.head_dim, 0, 0, 0, 0, 0.0, 0)
    k, idx, out, kc, vc = zipvl.zipvl_prefill_layer_host(desc, layer.q, layer.k, layer.v,
                                                         layer.probe_pos, layer.tau)
    r = gpu_pipeline(zipvl, layer)
    assert k == r["k"] and np.array_equal(idx.numpy(), r["idx"])
    assert torch.equal(out, r["out"].cpu())
    assert torch.equal(kc[:k], r["kc"][:k].cpu()) and torch.equal(vc[:k], r["vc"][:k].cpu())
    # the call keeps its device scratch in a pool of the library's own; releasing it is always
    # allowed and the next call simply allocates again
    zipvl.zipvl_release_host_scratch()
    k2, idx2, out2, _, _ = zipvl.zipvl_prefill_layer_host(desc, layer.q, layer.k, layer.v,
                                                          layer.probe_pos, layer.tau)
    assert k2 == k and torch.equal(idx2, idx) and torch.equal(out2, out)
    zipvl.zipvl_release_host_scratch()


@pytest.mark.parametrize("name", ["llava7b_small_bf16", "video_gqa_small", "tiny_fp32"])
def test_layer_step_host_entry_point_adds_a_decode_step(zipvl, name):
    """Algorithm 1 and one step of Algorithm 2 from host buffers in one call: the prefill
    results are those of zipvl_prefill_layer_host, the decode output is the oracle's on the
    compacted cache with the new token appended."""
    layer = CASES[name]()
    Hq, Hkv, d = layer.n_q_heads, layer.n_kv_heads, layer.head_dim
    code = {torch.bfloat16: zipvl.ZIPVL_BF16, torch.float32: zipvl.ZIPVL_F32}[layer.q.dtype]
    desc = zipvl.zipvl_layer(layer.L, Hq, Hkv, d, code, 0, 0, 0, 0.0, 0)
    g = torch.Generator().manual_seed(17)
    qn = torch.randn(1, Hq, d, generator=g).to(layer.q.dtype)
    kn = torch.randn(1, Hkv, d, generator=g).to(layer.q.dtype)
    vn = torch.randn(1, Hkv, d, generator=g).to(layer.q.dtype)
    k, idx, out, kc, vc, dec = zipvl.zipvl_layer_step_host(desc, layer.q, layer.k, layer.v, layer.probe_pos,
                                                           layer.tau, qn, kn, vn)
    k0, idx0, out0, kc0, vc0 = zipvl.zipvl_prefill_layer_host(desc, layer.q, layer.k, layer.v,
                                                              layer.probe_pos, layer.tau)
    assert k == k0 and torch.equal(idx, idx0) and torch.equal(out, out0)
    assert torch.equal(kc[:k], kc0[:k]) and torch.equal(vc[:k], vc0[:k])
    T = idx[:k].long()
    ko = np.concatenate([to_np(layer.k[T]).reshape(-1), np.zeros(Hkv * d, np.float32)])
    vo = np.concatenate([to_np(layer.v[T]).reshape(-1), np.zeros(Hkv * d, np.float32)])
    seq = np.array([k], np.int32)
    ref = oracle.decode_step(to_np(qn), to_np(kn), to_np(vn), ko, vo, np.zeros(1, np.int64), seq, Hkv)
    check_attention(to_np(dec), ref, layer.q.dtype)


def test_layer_step_replays_from_a_cuda_graph(zipvl):
    """score -> select -> fused prefill + compaction -> decode captured once into a CUDA
    graph (k stays on the device, nothing synchronises) and replayed on new inputs: the
    replays must equal eager execution bit for bit."""
    layers = [W.heavy_key_layer(L_visual=1150, L_text=64, H=8, seed=31 + s, probe_seed=77) for s in range(2)]
    L, H, d = layers[0].L, 8, 128
    q, k, v = (torch.empty_like(layers[0].q, device=DEV) for _ in range(3))
    probe = layers[0].probe_pos.to(DEV)
    desc = zipvl.layer_desc(q, k)
    i32 = torch.int32
    acc, norm = (torch.empty(L, dtype=torch.float32, device=DEV) for _ in range(2))
    k_dev, seq = torch.zeros(1, dtype=i32, device=DEV), torch.zeros(1, dtype=i32, device=DEV)
    idx = torch.empty(L, dtype=i32, device=DEV)
    out = torch.empty_like(q)
    cap = L + 8
    kc = torch.zeros(cap, H, d, dtype=q.dtype, device=DEV)
    vc = torch.zeros_like(kc)
    st = status_word()
    ws_s = zipvl.workspace(zipvl.zipvl_workspace_bytes(zipvl.OP_SCORE, desc, probe.numel()), DEV)
    ws_sel = zipvl.workspace(zipvl.zipvl_workspace_bytes(zipvl.OP_SELECT, desc), DEV)
    ws_p = zipvl.workspace(zipvl.zipvl_workspace_bytes(zipvl.OP_SPARSE_PREFILL, desc), DEV)
    ddesc = zipvl.zipvl_decode_desc(1, H, H, d, zipvl.ZIPVL_BF16, 0.0)
    dl = zipvl.zipvl_layer(cap, H, H, d, zipvl.ZIPVL_BF16, 0, 0, 0, 0.0, 0)
    ws_d = zipvl.workspace(zipvl.zipvl_workspace_bytes(zipvl.OP_DECODE, dl, 0, 1), DEV)
    g = torch.Generator().manual_seed(5)
    qn, kn, vn = (torch.randn(1, H, d, generator=g).bfloat16().to(DEV) for _ in range(3))
    off, capt = torch.zeros(1, dtype=torch.int64, device=DEV), torch.full((1,), cap, dtype=i32, device=DEV)
    dout = torch.empty(1, H, d, dtype=q.dtype, device=DEV)

    def step():
        zipvl.zipvl_score(desc, q, k, probe, acc=acc, norm=norm, ws=ws_s, status=st)
        zipvl.zipvl_select(acc, norm, layers[0].tau, k_out=k_dev, idx=idx, ws=ws_sel, status=st)
        zipvl.zipvl_sparse_prefill_compact(desc, q, k, v, idx, k_dev, L, kc, vc, cap, out=out, len_out=seq,
                                           ws=ws_p, status=st)
        zipvl.zipvl_decode(ddesc, qn, kn, vn, kc, vc, off, capt, seq, cap, out=dout, ws=ws_d, status=st)

    def load(layer):
        q.copy_(layer.q), k.copy_(layer.k), v.copy_(layer.v)

    eager = []
    for layer in layers:
        load(layer)
        step()
        torch.cuda.synchronize()
        eager.append([t.clone() for t in (acc, idx, k_dev, out, kc, vc, seq, dout)])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        load(layers[0])
        step()                                   # warm-up on the capture stream
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)
    for rep in range(2):
        for layer, ref in zip(layers, eager):
            load(layer)
            graph.replay()
            torch.cuda.synchronize()
            n_rows = int(ref[6].item())          # kept rows + the appended one; later rows are stale
            for j, (got, want) in enumerate(zip((acc, idx, k_dev, out, kc, vc, seq, dout), ref)):
                if j in (4, 5):
                    got, want = got[:n_rows], want[:n_rows]
                assert torch.equal(got, want), j
    assert int(st.item()) == 0


@pytest.mark.parametrize("kernel", ["tc", "tcp"])
def test_grouped_query_decode_steps_replay_from_a_cuda_graph(zipvl, monkeypatch, kernel):
    """Four decode steps with appends on grouped query heads, captured once into a CUDA graph
    (lengths live on the device, each step is a programmatic dependent of the one before) and
    replayed from reset lengths: the replays must equal eager execution bit for bit -- outputs,
    lengths and the appended cache rows."""
    monkeypatch.setenv("ZIPVL_DECODE_KERNEL", kernel)
    lens, Hq, Hkv, d, steps = [700, 129, 2600, 1], 14, 2, 128, 4
    B = len(lens)
    kc, vc, off, cap = build_caches(lens, Hkv, d, torch.bfloat16, steps, seed=77)
    g = torch.Generator().manual_seed(78)
    qs = torch.randn(steps, B, Hq, d, generator=g).bfloat16().to(DEV)
    kn = torch.randn(steps, B, Hkv, d, generator=g).bfloat16().to(DEV)
    vn = torch.randn(steps, B, Hkv, d, generator=g).bfloat16().to(DEV)
    desc = zipvl.zipvl_decode_desc(B, Hq, Hkv, d, zipvl.ZIPVL_BF16, 0.0)
    max_len = max(lens) + steps
    dl = zipvl.zipvl_layer(max_len, Hq, Hkv, d, zipvl.ZIPVL_BF16, 0, 0, 0, 0.0, 0)
    ws = zipvl.workspace(zipvl.zipvl_workspace_bytes(zipvl.OP_DECODE, dl, 0, B), DEV)
    kc_d, vc_d, off_d, cap_d = kc.to(DEV), vc.to(DEV), off.to(DEV), cap.to(DEV)
    seq0 = torch.tensor(lens, dtype=torch.int32, device=DEV)
    seq = seq0.clone()
    outs = torch.empty(steps, B, Hq, d, dtype=torch.bfloat16, device=DEV)
    st = status_word()

    def run():
        for s in range(steps):
            zipvl.zipvl_decode(desc, qs[s], kn[s], vn[s], kc_d, vc_d, off_d, cap_d, seq, max_len,
                               out=outs[s], ws=ws, status=st)

    run()
    torch.cuda.synchronize()
    want = (outs.clone(), seq.clone(), kc_d.clone(), vc_d.clone())
    # the eager run against the oracle, step by step
    ko, vo, seqo = to_np(kc).copy(), to_np(vc).copy(), np.array(lens, np.int32)
    for s in range(steps):
        ref = oracle.decode_step(to_np(qs[s].cpu()), to_np(kn[s].cpu()), to_np(vn[s].cpu()), ko, vo,
                                 off.numpy(), seqo, Hkv)
        check_attention(to_np(want[0][s].cpu()), ref, torch.bfloat16)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        seq.copy_(seq0)
        run()                                    # warm-up on the capture stream
        seq.copy_(seq0)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            run()
    torch.cuda.current_stream().wait_stream(side)
    for rep in range(3):
        seq.copy_(seq0)
        outs.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(outs, want[0]) and torch.equal(seq, want[1])
        assert torch.equal(kc_d, want[2]) and torch.equal(vc_d, want[3])
    assert int(st.item()) == 0


@pytest.mark.parametrize("kernel", ["tc", "tcp"])
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_grouped_query_decode_random_batches(zipvl, monkeypatch, kernel, seed):
    """Random ragged batches on the tensor-core decode kernels: empty and one-row requests next to
    requests of several tiles, group sizes from 3 to 16, with and without a new token, two steps
    each, against the oracle.  (Short and long work items side by side are what the persistent
    kernel's segment hand-over has to get right.)"""
    monkeypatch.setenv("ZIPVL_DECODE_KERNEL", kernel)
    rng = np.random.default_rng(1000 + seed)
    for trial in range(3):
        G = int(rng.choice([3, 4, 7, 8, 16]))
        Hkv = int(rng.choice([1, 2, 4]))
        Hq, d = G * Hkv, 128
        B = int(rng.integers(1, 7))
        lens = [int(x) for x in rng.choice([0, 1, 5, 127, 128, 129, 300, 777, 1500, 2600, 4100], size=B)]
        dtype = torch.bfloat16 if trial % 2 == 0 else torch.float16
        code = zipvl.ZIPVL_BF16 if dtype == torch.bfloat16 else zipvl.ZIPVL_F16
        kc, vc, off, cap = build_caches(lens, Hkv, d, dtype, 2, seed=seed * 10 + trial)
        g = torch.Generator().manual_seed(seed * 100 + trial)
        desc = zipvl.zipvl_decode_desc(B, Hq, Hkv, d, code, 0.0)
        kc_d, vc_d, off_d, cap_d = kc.to(DEV), vc.to(DEV), off.to(DEV), cap.to(DEV)
        seq_d = torch.tensor(lens, dtype=torch.int32, device=DEV)
        ko, vo, seqo = kc.float().numpy().copy(), vc.float().numpy().copy(), np.array(lens, np.int32)
        st = status_word()
        max_len = max(lens) + 2
        for step in range(2):
            q = torch.randn(B, Hq, d, generator=g).to(dtype)
            append = bool((seed + trial + step) % 2 == 0)
            kn = torch.randn(B, Hkv, d, generator=g).to(dtype) if append else None
            vn = torch.randn(B, Hkv, d, generator=g).to(dtype) if append else None
            out = zipvl.zipvl_decode(desc, q.to(DEV), None if kn is None else kn.to(DEV),
                                     None if vn is None else vn.to(DEV), kc_d, vc_d, off_d, cap_d, seq_d,
                                     max_len, status=st)
            ref = oracle.decode_step(to_np(q), None if kn is None else to_np(kn),
                                     None if vn is None else to_np(vn), ko, vo, off.numpy(), seqo, Hkv)
            check_attention(to_np(out), ref, dtype)
            assert np.array_equal(seq_d.cpu().numpy(), seqo)
        assert st.item() == 0
        assert np.array_equal(kc_d.float().cpu().numpy(), ko) and np.array_equal(vc_d.float().cpu().numpy(), vo)
