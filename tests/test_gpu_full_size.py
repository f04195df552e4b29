"""GPU parity at the paper-shaped sizes, in the launch configuration bench.py
times: the LLaVA-Next-7B layer, layers of the 13B 40-layer stack, the long-video
GQA layer and a ragged decode batch on compacted caches.  The oracle checks the
scores in full, the selection exactly (on the GPU's own scores), and sampled
rows of the attention outputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_08584_b200 import workloads as W
from parity import check_attention, check_scores, check_select, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_layer(z, layer, n_rows=48, seed=0, attention=True):
    q, k, v, probe = (t.to(DEV) for t in (layer.q, layer.k, layer.v, layer.probe_pos))
    desc = z.layer_desc(q, k)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    acc, norm = z.zipvl_score(desc, q, k, probe, status=st)
    k_dev, idx = z.zipvl_select(acc, norm, layer.tau, status=st)
    out = z.zipvl_sparse_prefill(desc, q, k, v, idx, k_dev, layer.L, status=st)   # padded, k_max = L
    kc, vc = torch.zeros_like(k), torch.zeros_like(v)
    n = z.zipvl_compact_kv(desc, k, v, idx, k_dev, layer.L, kc, vc, layer.L, status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    kk = int(k_dev.item())
    qf, kf, vf = to_np(layer.q), to_np(layer.k), to_np(layer.v)
    # scores, in full
    acc_ref, S = oracle.probe_scores(qf, kf, layer.probe_pos.numpy())
    norm_ref, _ = oracle.normalise(acc_ref, layer.probe_pos.numpy(), layer.n_q_heads)
    err = check_scores(acc.cpu().numpy(), norm.cpu().numpy(), acc_ref, norm_ref, S)
    # selection, exact on the GPU's own scores
    idx_h = idx.cpu().numpy()
    check_select(kk, idx_h, acc.cpu().numpy().astype(np.float64),
                 norm.cpu().numpy().astype(np.float64), layer.tau)
    # and against the pure oracle within the measured score error
    check_select(kk, idx_h, acc_ref, norm_ref, layer.tau, eps=max(1e-6, 4 * err))
    T = idx_h[:kk]
    if not attention:
        return kk
    # attention: sampled rows of T (first, last, tile edges and a seeded sample)
    rng = np.random.default_rng(seed)
    edges = [r for r in (0, 1, 127, 128, 255, 256, 257, kk - 129, kk - 2, kk - 1) if 0 <= r < kk]
    rows = np.unique(np.concatenate([edges, rng.integers(0, kk, n_rows)])).astype(np.int32)
    ref = oracle.sparse_prefill(qf, kf, vf, T, rows=rows)
    out_h = out.float().cpu().numpy()
    check_attention(out_h[T[rows]], ref, layer.q.dtype)
    U = np.setdiff1d(np.arange(layer.L), T)
    assert not out_h[U].any(), "rows of dropped tokens must be zero"
    # compaction, bit-exact
    assert int(n.item()) == kk
    Tl = torch.from_numpy(T).long()
    assert torch.equal(kc[:kk].cpu(), layer.k[Tl]) and torch.equal(vc[:kk].cpu(), layer.v[Tl])
    # the fused call (attention + compaction in one kernel, what bench.py times) gives the same bits
    kc2, vc2 = torch.zeros_like(k), torch.zeros_like(v)
    out2, n2 = z.zipvl_sparse_prefill_compact(desc, q, k, v, idx, k_dev, layer.L, kc2, vc2, layer.L, status=st)
    torch.cuda.synchronize()
    assert st.item() == 0 and int(n2.item()) == kk
    assert torch.equal(out2, out) and torch.equal(kc2[:kk], kc[:kk]) and torch.equal(vc2[:kk], vc[:kk])
    return kk


def test_llava_next_7b_layer_full_size(zipvl):
    layer = W.heavy_key_layer()          # L 2944, 32 heads x 128, bf16, tau 0.97
    k = run_layer(zipvl, layer)
    assert 0.5 * layer.L < k < layer.L


def test_llava_next_7b_layer_full_size_fp16(zipvl):
    layer = W.heavy_key_layer(dtype=torch.float16)     # the same layer stored as IEEE half
    run_layer(zipvl, layer, n_rows=32, seed=5)


def test_llava_next_13b_stack_all_forty_layers(zipvl):
    """Every layer of the 40-layer stack: scores in full and the selection (exact on the GPU's
    scores, and against the pure oracle within the measured score error); attention on sampled
    rows, compaction and the fused call for every fourth layer.  The per-layer budget is the
    point of the configuration, so it must vary widely."""
    ks = [run_layer(zipvl, W.stack_layer(i), n_rows=16, seed=i, attention=(i % 4 == 0 or i == 39))
          for i in range(40)]
    assert len(set(ks)) >= 30 and max(ks) > 3 * min(ks), f"per-layer k should vary widely: {ks}"


def test_llava_next_13b_layer_at_32k_tokens(zipvl):
    """The 13B-shaped layer at the first of the long input lengths the bench's long-context leg
    times (32768 tokens, 40 heads x 128): scores in full, the selection exactly, sampled rows
    of the attention, compaction and the fused call."""
    layer = W.heavy_key_layer(L_visual=32768 - 64, L_text=64, H=40, seed=W.BASE_SEED + 72, name="llava_next_13b_long")
    k = run_layer(zipvl, layer, n_rows=12, seed=3)
    assert 0.5 * layer.L < k < layer.L


def test_full_size_layer_repeated_on_a_side_stream(zipvl):
    """The whole chain (score, select, fused attention + compaction) three hundred times on a
    non-default stream, where every launch is a programmatic dependent of the one before
    and the attention grid runs in two waves: no device status, and every repetition gives
    the bits of the first."""
    layer = W.heavy_key_layer()
    q, k, v, probe = (t.to(DEV) for t in (layer.q, layer.k, layer.v, layer.probe_pos))
    desc = zipvl.layer_desc(q, k)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    out, kc, vc = torch.empty_like(q), torch.zeros_like(k), torch.zeros_like(v)
    first = None
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        acc, norm = zipvl.zipvl_score(desc, q, k, probe, status=st)
        k_dev, idx = zipvl.zipvl_select(acc, norm, layer.tau, status=st)
        for it in range(300):
            zipvl.zipvl_score(desc, q, k, probe, acc=acc, norm=norm, status=st)
            zipvl.zipvl_select(acc, norm, layer.tau, k_out=k_dev, idx=idx, status=st)
            zipvl.zipvl_sparse_prefill_compact(desc, q, k, v, idx, k_dev, layer.L, kc, vc, layer.L,
                                               out=out, status=st)
            if it == 0:
                side.synchronize()
                first = (out.clone(), kc.clone(), vc.clone(), idx.clone())
        side.synchronize()
    assert st.item() == 0
    assert torch.equal(out, first[0]) and torch.equal(kc, first[1]) and torch.equal(vc, first[2])
    assert torch.equal(idx, first[3])


@pytest.mark.parametrize("tau", [0.95, 0.99])
def test_long_video_gqa_full_size(zipvl, tau):
    layer = W.video_layer(tau=tau)       # L 18432, 28 / 4 heads
    k = run_layer(zipvl, layer, n_rows=24)
    assert k > 0.8 * layer.L


def test_ragged_decode_on_compacted_caches(zipvl):
    """Requests of different context lengths are scored, selected and compacted on
    the GPU, then decoded as one ragged batch; compared step by step with the
    oracle on the same compacted caches, and once on the dense caches."""
    z = zipvl
    batch = W.decode_batch(B=5, ctx_min=4096, ctx_max=9000, H=32, d=128, steps=3)
    B, Hq, d, steps = 5, 32, 128, 3
    row = Hq * d
    ks, kcs, vcs = [], [], []
    for lay in batch.layers:
        q, k, v, probe = (t.to(DEV) for t in (lay.q, lay.k, lay.v, lay.probe_pos))
        desc = z.layer_desc(q, k)
        acc, norm = z.zipvl_score(desc, q, k, probe)
        k_dev, idx = z.zipvl_select(acc, norm, batch.tau)
        kb = int(k_dev.item())
        kc = torch.zeros(kb + steps, Hq, d, dtype=torch.bfloat16, device=DEV)
        vc = torch.zeros_like(kc)
        z.zipvl_compact_kv(desc, k, v, idx, k_dev, lay.L, kc, vc, kb + steps)
        T = idx[:kb].long()
        assert torch.equal(kc[:kb], k[T]) and torch.equal(vc[:kb], v[T])
        ks.append(kb)
        kcs.append(kc.reshape(-1))
        vcs.append(vc.reshape(-1))
    assert len(set(ks)) == B
    for name, k_list, v_list, lens in (("compacted", kcs, vcs, ks),
                                       ("dense", [torch.cat([l.k.to(DEV).reshape(-1), torch.zeros(steps * row, dtype=torch.bfloat16, device=DEV)]) for l in batch.layers],
                                        [torch.cat([l.v.to(DEV).reshape(-1), torch.zeros(steps * row, dtype=torch.bfloat16, device=DEV)]) for l in batch.layers],
                                        batch.ctx_lens)):
        caps = [n + steps for n in lens]
        off = torch.tensor(np.concatenate([[0], np.cumsum([c * row for c in caps[:-1]])]), dtype=torch.int64)
        kcache, vcache = torch.cat(k_list), torch.cat(v_list)
        seq = torch.tensor(lens, dtype=torch.int32, device=DEV)
        ko, vo = kcache.float().cpu().numpy().copy(), vcache.float().cpu().numpy().copy()
        seqo = np.array(lens, np.int32)
        desc = z.zipvl_decode_desc(B, Hq, Hq, d, z.ZIPVL_BF16, 0.0)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        n_steps = steps if name == "compacted" else 1
        for s in range(n_steps):
            qn, kn, vn = batch.q_steps[s], batch.k_steps[s], batch.v_steps[s]
            out = z.zipvl_decode(desc, qn.to(DEV), kn.to(DEV), vn.to(DEV), kcache, vcache,
                                 off.to(DEV), torch.tensor(caps, dtype=torch.int32, device=DEV),
                                 seq, max(caps), status=st)
            ref = oracle.decode_step(to_np(qn), to_np(kn), to_np(vn), ko, vo, off.numpy(), seqo, Hq)
            check_attention(to_np(out), ref, torch.bfloat16)
            assert np.array_equal(seq.cpu().numpy(), seqo)
        assert st.item() == 0


def test_batched_decode_full_size_compacted_and_dense(zipvl):
    """The batched-decode configuration at the size bench.py times: 16 requests with contexts
    drawn from 4096..32768, 32 heads x 128, bf16, host-generated data.  Each request is scored,
    selected and compacted on the GPU (compaction checked bit for bit against K[T], V[T]); then
    four decode steps over the compacted caches and four over the dense ones, every output of
    every request and head against the oracle's decode step."""
    z = zipvl
    B, H, d, steps = 16, 32, 128, 4
    batch = W.decode_batch(B=B, ctx_min=4096, ctx_max=32768, H=H, d=d, steps=steps)
    row = H * d
    assert min(batch.ctx_lens) >= 4096 and max(batch.ctx_lens) > 20000
    ks, comp_k, comp_v = [], [], []
    for lay in batch.layers:
        q, k, v, probe = (t.to(DEV) for t in (lay.q, lay.k, lay.v, lay.probe_pos))
        desc = z.layer_desc(q, k)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        acc, norm = z.zipvl_score(desc, q, k, probe, status=st)
        k_dev, idx = z.zipvl_select(acc, norm, batch.tau, status=st)
        kb = int(k_dev.item())
        kc = torch.zeros(kb + steps, H, d, dtype=torch.bfloat16, device=DEV)
        vc = torch.zeros_like(kc)
        z.zipvl_compact_kv(desc, k, v, idx, k_dev, lay.L, kc, vc, kb + steps, status=st)
        T = idx[:kb].long().cpu()
        assert st.item() == 0
        assert torch.equal(kc[:kb].cpu(), lay.k[T]) and torch.equal(vc[:kb].cpu(), lay.v[T])
        check_select(kb, idx.cpu().numpy(), acc.cpu().numpy().astype(np.float64),
                     norm.cpu().numpy().astype(np.float64), batch.tau)
        ks.append(kb)
        comp_k.append(kc.reshape(-1).cpu())
        comp_v.append(vc.reshape(-1).cpu())
        lay.q = None                                  # the context queries are not needed again
        del q, k, v, kc, vc
    assert len(set(ks)) == B
    pad = torch.zeros(steps * row, dtype=torch.bfloat16)
    dense_k = [torch.cat([l.k.reshape(-1), pad]) for l in batch.layers]
    dense_v = [torch.cat([l.v.reshape(-1), pad]) for l in batch.layers]
    ddesc = z.zipvl_decode_desc(B, H, H, d, z.ZIPVL_BF16, 0.0)
    for name, k_list, v_list, lens in (("compacted", comp_k, comp_v, ks),
                                       ("dense", dense_k, dense_v, batch.ctx_lens)):
        caps = [n + steps for n in lens]
        off = np.concatenate([[0], np.cumsum([c * row for c in caps[:-1]])]).astype(np.int64)
        kcache, vcache = torch.cat(k_list), torch.cat(v_list)
        ko, vo = kcache.float().numpy(), vcache.float().numpy()     # the oracle's own copies
        kcache, vcache = kcache.to(DEV), vcache.to(DEV)
        seq = torch.tensor(lens, dtype=torch.int32, device=DEV)
        seqo = np.array(lens, np.int32)
        capt = torch.tensor(caps, dtype=torch.int32, device=DEV)
        off_d = torch.from_numpy(off).to(DEV)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        for s_ in range(steps):
            qn, kn, vn = batch.q_steps[s_], batch.k_steps[s_], batch.v_steps[s_]
            out = z.zipvl_decode(ddesc, qn.to(DEV), kn.to(DEV), vn.to(DEV), kcache, vcache, off_d, capt,
                                 seq, max(caps), status=st)
            ref = oracle.decode_step(to_np(qn), to_np(kn), to_np(vn), ko, vo, off, seqo, H)
            check_attention(to_np(out), ref, torch.bfloat16)
            assert np.array_equal(seq.cpu().numpy(), seqo)
        assert st.item() == 0
        # the appended rows went into the caches bit for bit
        assert np.array_equal(kcache.float().cpu().numpy(), ko) and np.array_equal(vcache.float().cpu().numpy(), vo)
        del kcache, vcache, ko, vo


@pytest.mark.parametrize("paged", [False, True])
def test_grouped_query_decode_full_size(zipvl, paged):
    """The grouped-query decode configuration bench.py times (16 requests of 6000 to 30000 kept
    rows, 28 query heads on 4 kv heads, head_dim 128, bf16), on the kernel the library picks at
    that size: three steps with appended tokens, every output of every request and head, the
    lengths and the appended rows against the oracle.  Once on contiguous caches, once on a
    paged pool whose pages are dealt out in a shuffled order."""
    z = zipvl
    B, Hq, Hkv, d, steps = 16, 28, 4, 128, 3
    row = Hkv * d
    g = torch.Generator().manual_seed(4242)
    lens = torch.randint(6000, 30001, (B,), generator=g).tolist()
    caps = [n + steps for n in lens]
    page_rows = 128
    if not paged:
        off = np.concatenate([[0], np.cumsum([c * row for c in caps[:-1]])]).astype(np.int64)
        total_rows = sum(caps)
    else:
        pages_of = [(c + page_rows - 1) // page_rows for c in caps]
        n_pages = sum(pages_of)
        perm = torch.randperm(n_pages, generator=g).numpy().astype(np.int32)
        table = np.full((B, max(pages_of)), -1, np.int32)
        at = 0
        for b, n in enumerate(pages_of):
            table[b, :n] = perm[at: at + n]
            at += n
        total_rows = n_pages * page_rows
    kc = torch.zeros(total_rows * row, dtype=torch.bfloat16)
    vc = torch.zeros(total_rows * row, dtype=torch.bfloat16)

    def rows_of(b, n):               # element offsets of request b's first n rows
        if not paged:
            return off[b] + np.arange(n, dtype=np.int64) * row
        r = np.arange(n, dtype=np.int64)
        return (table[b, r // page_rows].astype(np.int64) * page_rows + r % page_rows) * row

    for b, n in enumerate(lens):
        kv = torch.randn(2, n, row, generator=g).to(torch.bfloat16)
        at = torch.from_numpy(rows_of(b, n))[:, None] + torch.arange(row)[None, :]
        kc[at.reshape(-1)] = kv[0].reshape(-1)
        vc[at.reshape(-1)] = kv[1].reshape(-1)
    # the oracle works on contiguous per-request caches of its own
    o_off = np.concatenate([[0], np.cumsum([c * row for c in caps[:-1]])]).astype(np.int64)
    ko = np.zeros(sum(caps) * row, np.float32)
    vo = np.zeros(sum(caps) * row, np.float32)
    for b, n in enumerate(lens):
        at = (torch.from_numpy(rows_of(b, n))[:, None] + torch.arange(row)[None, :]).reshape(-1)
        ko[o_off[b]: o_off[b] + n * row] = kc[at].float().numpy()
        vo[o_off[b]: o_off[b] + n * row] = vc[at].float().numpy()
    seqo = np.array(lens, np.int32)
    kc_d, vc_d = kc.to(DEV), vc.to(DEV)
    seq = torch.tensor(lens, dtype=torch.int32, device=DEV)
    capt = torch.tensor(caps, dtype=torch.int32, device=DEV)
    desc = z.zipvl_decode_desc(B, Hq, Hkv, d, z.ZIPVL_BF16, 0.0)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    for s_ in range(steps):
        qn = torch.randn(B, Hq, d, generator=g).to(torch.bfloat16)
        kn = torch.randn(B, Hkv, d, generator=g).to(torch.bfloat16)
        vn = torch.randn(B, Hkv, d, generator=g).to(torch.bfloat16)
        if not paged:
            out = z.zipvl_decode(desc, qn.to(DEV), kn.to(DEV), vn.to(DEV), kc_d, vc_d,
                                 torch.from_numpy(off).to(DEV), capt, seq, max(caps), status=st)
        else:
            out = z.zipvl_decode_paged(desc, qn.to(DEV), kn.to(DEV), vn.to(DEV),
                                       kc_d.view(n_pages, page_rows, Hkv, d), vc_d.view(n_pages, page_rows, Hkv, d),
                                       torch.from_numpy(table).to(DEV), capt, seq, max(caps), status=st)
        ref = oracle.decode_step(to_np(qn), to_np(kn), to_np(vn), ko, vo, o_off, seqo, Hkv)
        check_attention(to_np(out), ref, torch.bfloat16)
        assert np.array_equal(seq.cpu().numpy(), seqo)
    assert st.item() == 0
    # the appended rows went into the caches bit for bit
    kh, vh = kc_d.float().cpu().numpy(), vc_d.float().cpu().numpy()
    for b in range(B):
        at = (rows_of(b, lens[b] + steps)[:, None] + np.arange(row)[None, :]).reshape(-1)
        assert np.array_equal(kh[at], ko[o_off[b]: o_off[b] + (lens[b] + steps) * row])
        assert np.array_equal(vh[at], vo[o_off[b]: o_off[b] + (lens[b] + steps) * row])


@pytest.mark.parametrize("kernel", ["tc", "tcp"])
def test_grouped_query_decode_many_steps_on_a_side_stream(zipvl, monkeypatch, kernel):
    """Two hundred decode steps with appends per shape on a non-default stream, every launch a
    programmatic dependent of the one before, on both tensor-core kernels: no wait runs out (status
    word), the lengths advance by one per step, and the last step's output matches the oracle."""
    z = zipvl
    monkeypatch.setenv("ZIPVL_DECODE_KERNEL", kernel)
    rng = np.random.default_rng(11)
    for trial, (Hq, Hkv, d) in enumerate([(28, 4, 128), (32, 2, 64), (16, 8, 96)]):
        B, steps = int(rng.integers(3, 12)), 200
        lens = [int(x) for x in rng.integers(0, 5000, B)]
        row = Hkv * d
        caps = [n + steps for n in lens]
        g = torch.Generator().manual_seed(trial)
        kc = torch.randn(sum(caps) * row, generator=g).to(torch.bfloat16)
        vc = torch.randn(sum(caps) * row, generator=g).to(torch.bfloat16)
        off = np.concatenate([[0], np.cumsum([c * row for c in caps[:-1]])]).astype(np.int64)
        q = torch.randn(B, Hq, d, generator=g).to(torch.bfloat16)
        kn = torch.randn(B, Hkv, d, generator=g).to(torch.bfloat16)
        vn = torch.randn(B, Hkv, d, generator=g).to(torch.bfloat16)
        kc_d, vc_d, q_d, kn_d, vn_d = (t.to(DEV) for t in (kc, vc, q, kn, vn))
        off_d = torch.from_numpy(off).to(DEV)
        capt = torch.tensor(caps, dtype=torch.int32, device=DEV)
        seq = torch.tensor(lens, dtype=torch.int32, device=DEV)
        desc = z.zipvl_decode_desc(B, Hq, Hkv, d, z.ZIPVL_BF16, 0.0)
        lay = z.zipvl_layer(max(caps), Hq, Hkv, d, z.ZIPVL_BF16, 0, 0, 0, 0.0, 0)
        ws = z.workspace(z.zipvl_workspace_bytes(z.OP_DECODE, lay, 0, B), DEV)
        out = torch.empty_like(q_d)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(steps):
                z.zipvl_decode(desc, q_d, kn_d, vn_d, kc_d, vc_d, off_d, capt, seq, max(caps), out=out, ws=ws,
                               status=st)
        side.synchronize()
        assert st.item() == 0
        assert np.array_equal(seq.cpu().numpy(), np.array(lens) + steps)
        # the oracle's view of the last step: the caches as the GPU left them, one row short
        ko, vo = kc_d.float().cpu().numpy(), vc_d.float().cpu().numpy()
        seqo = np.array(lens, np.int32) + steps - 1
        ref = oracle.decode_step(to_np(q), to_np(kn), to_np(vn), ko, vo, off, seqo, Hkv)
        check_attention(to_np(out), ref, torch.bfloat16)
