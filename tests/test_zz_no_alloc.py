"""zipvl_decode_noalloc: the decode step for callers that cannot allocate device
memory (no workspace argument; the scratch is a fixed array inside the library).

Checked through the C ABI against zipvl_decode on the same inputs (bit for bit:
the two entry points run the same kernels) and against the CPU oracle's decode
step, two calls in a row (the second call finds the previous call's data in the
shared scratch).
This file sorts last on purpose: a run that stops at the first failure has
already run every other test.  It also passes when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle
from parity import check_attention, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _caches(lens, Hkv, d, extra, seed):
    g = torch.Generator().manual_seed(seed)
    cap = [n + extra for n in lens]
    row = Hkv * d
    off = np.concatenate([[0], np.cumsum([c * row for c in cap[:-1]])]).astype(np.int64)
    kc = torch.zeros(sum(cap) * row, dtype=torch.bfloat16)
    vc = torch.zeros_like(kc)
    for b, n in enumerate(lens):
        kc[off[b]: off[b] + n * row] = torch.randn(n * row, generator=g).bfloat16()
        vc[off[b]: off[b] + n * row] = torch.randn(n * row, generator=g).bfloat16()
    return kc, vc, torch.from_numpy(off), torch.tensor(cap, dtype=torch.int32)


def test_noalloc_decode_matches_decode_twice_in_a_row(zipvl):
    lens, Hq, Hkv, d = [700, 33, 1500, 257], 8, 2, 128
    B = len(lens)
    kc, vc, off, cap = _caches(lens, Hkv, d, extra=4, seed=123)
    desc = zipvl.zipvl_decode_desc(B, Hq, Hkv, d, zipvl.ZIPVL_BF16, 0.0)
    max_len = max(lens) + 4
    g = torch.Generator().manual_seed(7)
    # two independent copies of the caches: one per entry point
    state = []
    for _ in range(2):
        state.append(dict(kc=kc.to(DEV), vc=vc.to(DEV),
                          seq=torch.tensor(lens, dtype=torch.int32, device=DEV)))
    off_d, cap_d = off.to(DEV), cap.to(DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    # the oracle's own copy of the caches (float32 holds bf16 exactly)
    ko, vo, seqo = to_np(kc).copy(), to_np(vc).copy(), np.array(lens, np.int32)
    for call in range(2):
        q = torch.randn(B, Hq, d, generator=g).bfloat16()
        kn = torch.randn(B, Hkv, d, generator=g).bfloat16()
        vn = torch.randn(B, Hkv, d, generator=g).bfloat16()
        ref = zipvl.zipvl_decode(desc, q.to(DEV), kn.to(DEV), vn.to(DEV), state[0]["kc"], state[0]["vc"],
                                 off_d, cap_d, state[0]["seq"], max_len, status=st)
        out = torch.full((B, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
        zipvl.zipvl_decode_noalloc(desc, q.to(DEV), kn.to(DEV), vn.to(DEV), state[1]["kc"], state[1]["vc"],
                                   off_d, cap_d, state[1]["seq"], max_len, out, status=st)
        torch.cuda.synchronize()
        # same kernels, same chunking, same order of operations: the same bits
        assert torch.equal(out, ref)
        # and the right answer: Algorithm 2 by the oracle on its own copy of the caches
        want = oracle.decode_step(to_np(q), to_np(kn), to_np(vn), ko, vo, off.numpy(), seqo, Hkv)
        check_attention(to_np(out), want, torch.bfloat16)
        assert np.array_equal(state[1]["seq"].cpu().numpy(), seqo)
        assert torch.equal(state[0]["seq"], state[1]["seq"])
        assert torch.equal(state[0]["kc"], state[1]["kc"]) and torch.equal(state[0]["vc"], state[1]["vc"])
    assert st.item() == 0
    assert state[1]["seq"].tolist() == [n + 2 for n in lens]


def test_noalloc_decode_refuses_sizes_beyond_its_scratch(zipvl):
    """A problem whose partial results would not fit the built-in scratch is refused on the
    host with a clear message.  The buffers handed over are real (small) device tensors, so
    nothing depends on the order of the library's checks."""
    B, H, d = 16, 32, 128
    desc = zipvl.zipvl_decode_desc(B, H, H, d, zipvl.ZIPVL_BF16, 0.0)
    q = torch.zeros(B, H, d, dtype=torch.bfloat16, device=DEV)
    kc = torch.zeros(B * 8 * H * d, dtype=torch.bfloat16, device=DEV)      # 8 rows per request
    vc = torch.zeros_like(kc)
    off = (torch.arange(B, dtype=torch.int64) * 8 * H * d).to(DEV)
    cap = torch.full((B,), 8, dtype=torch.int32, device=DEV)
    seq = torch.full((B,), 3, dtype=torch.int32, device=DEV)
    out = torch.empty_like(q)
    with pytest.raises(zipvl.ZipvlError) as e:
        # max_len is only a bound the caller states; 32768 needs more scratch than there is
        zipvl.zipvl_decode_noalloc(desc, q, None, None, kc, vc, off, cap, seq, 32768, out)
    assert e.value.status == 3 and "scratch" in str(e.value)
    # the same buffers with an honest bound are served
    zipvl.zipvl_decode_noalloc(desc, q, None, None, kc, vc, off, cap, seq, 8, out)
    torch.cuda.synchronize()
    assert not out.float().abs().max().item() > 0      # all-zero values: the output is zero
