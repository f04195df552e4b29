"""Comparator rules shared by the GPU parity tests (CUDA path vs CPU oracle).

Tolerances (derived in the design notes):
  scores     fp32 accumulation of exact products + hardware exp2:
             relative 5e-5 where a_j > 1e-6*S, absolute 1e-7*S elsewhere;
  selection  exact, except members whose ranking score lies within a relative
             epsilon of the threshold value (ties), epsilon = 1e-6 when the
             oracle is fed the GPU's own scores;
  attention  bf16: max-abs 2e-2, mean-abs 2e-3; fp32: max-abs 1e-4, mean-abs 1e-5;
  compaction bit-exact.
"""
import numpy as np
import torch

import oracle

SCORE_RTOL = 5e-5
# IEEE half rounds P and the output to 11 bits instead of bfloat16's 8: a tighter bound
ATT_TOL = {torch.bfloat16: (2e-2, 2e-3), torch.float16: (4e-3, 4e-4), torch.float32: (1e-4, 1e-5)}


def to_np(t):
    """Stored values, exactly, as float32 numpy (bf16 and fp16 upcast losslessly)."""
    return t.detach().float().cpu().numpy()


def check_scores(acc_gpu, norm_gpu, acc_ref, norm_ref, S):
    acc_gpu, norm_gpu = acc_gpu.astype(np.float64), norm_gpu.astype(np.float64)
    big = acc_ref > 1e-6 * S
    rel = np.abs(acc_gpu[big] - acc_ref[big]) / acc_ref[big]
    assert rel.size == 0 or rel.max() <= SCORE_RTOL, f"acc rel err {rel.max():.3e}"
    small = ~big
    if small.any():
        assert np.abs(acc_gpu[small] - acc_ref[small]).max() <= 1e-7 * S
    # columns no probe can see are exactly zero on both sides
    assert np.all(acc_gpu[acc_ref == 0.0] == 0.0)
    nb = norm_ref > 0
    reln = np.abs(norm_gpu[nb & big] - norm_ref[nb & big]) / norm_ref[nb & big]
    assert reln.size == 0 or reln.max() <= SCORE_RTOL, f"norm rel err {reln.max():.3e}"
    return float(rel.max()) if rel.size else 0.0


def check_select(k_gpu, idx_gpu, acc, norm, tau, eps=1e-6, budget_metric=oracle.METRIC_ACC,
                 topk_metric=oracle.METRIC_NORM, fixed_k=0, keep_last=0):
    """acc / norm: the float64 scores the oracle selects from.  k may differ from
    the oracle only when a prefix sum sits within eps*S of the target; members may
    differ only among tokens whose ranking score is within eps (relative) of the
    threshold value."""
    L = len(acc)
    tau = float(np.float32(tau))      # the C ABI takes a float: both sides get the same number
    p, T, diag = oracle.select(acc, norm, tau, budget_metric, topk_metric, fixed_k)
    idx_gpu = np.asarray(idx_gpu)
    if keep_last > 0:
        # the final positions must all be in; what is left is compared as without the option
        # (positions the rule itself takes stay, the ones only the option added are removed)
        forced = np.arange(max(0, L - keep_last), L)
        Tg_all = idx_gpu[:k_gpu]
        assert np.all(idx_gpu[k_gpu:] == -1) and (k_gpu <= 1 or np.all(np.diff(Tg_all) > 0))
        assert np.all(np.isin(forced, Tg_all)), "a final position is missing"
        k_or, T_or, _ = oracle.select(acc, norm, tau, budget_metric, topk_metric, fixed_k, keep_last)
        added = np.setdiff1d(forced, T)                  # by the oracle's own rule-only set
        if k_gpu == k_or and np.array_equal(Tg_all, T_or):
            return k_or, T_or
        # ties at the threshold: strip the positions only the option can have added and
        # fall through to the tolerant comparison of the rule-only sets
        rule_only = np.setdiff1d(Tg_all, added)
        idx_gpu = np.concatenate([rule_only, np.full(L - len(rule_only), -1)]).astype(np.int64)
        k_gpu = len(rule_only)
    Tg = idx_gpu[:k_gpu]
    assert np.all(idx_gpu[k_gpu:] == -1), "tail of idx must be -1"
    assert len(Tg) == k_gpu and (k_gpu <= 1 or np.all(np.diff(Tg) > 0)), "idx not ascending"
    assert k_gpu >= 1 and Tg.min() >= 0 and Tg.max() < L
    if k_gpu != p:
        assert diag, "fixed_k must be honoured exactly"
        bm = acc if budget_metric == oracle.METRIC_ACC else norm
        srt = np.sort(bm)[::-1]
        C = np.cumsum(srt)
        lo, hi = min(p, k_gpu), max(p, k_gpu)
        # every prefix between the two answers must sit within eps*S of the target
        assert np.all(np.abs(C[lo - 1:hi] - diag["target"]) <= eps * diag["S"]), \
            f"k differs ({k_gpu} vs oracle {p}) outside the tie margin"
    rank = acc if topk_metric == oracle.METRIC_ACC else norm
    sym = np.setxor1d(Tg, T)
    if sym.size:
        # Tokens in descending rank (ties toward the smaller position).  Where k agrees the
        # sets may differ only among ties of the k-th value.  Where k differs (allowed above
        # only inside the tie margin of the budget) the extra members are exactly the tokens
        # ranked between the two answers -- again up to ties at either end.
        order = np.lexsort((np.arange(L), -rank))
        lo, hi = min(k_gpu, p), max(k_gpu, p)
        between = order[lo:hi]
        ends = [rank[order[lo - 1]], rank[order[hi - 1]]]
        tie = np.zeros(sym.size, bool)
        for thr in ends:
            tie |= np.abs(rank[sym] - thr) <= eps * max(thr, 1e-300)
        ok = tie | np.isin(sym, between)
        assert ok.all(), f"selected set differs outside ties: {sym[~ok][:8]}"
    return p, T


def check_attention(out_gpu, out_ref, dtype):
    max_tol, mean_tol = ATT_TOL[dtype]
    d = np.abs(out_gpu.astype(np.float64) - out_ref)
    assert np.isfinite(out_gpu).all()
    assert d.max() <= max_tol, f"max-abs {d.max():.3e} > {max_tol}"
    assert d.mean() <= mean_tol, f"mean-abs {d.mean():.3e} > {mean_tol}"
    return float(d.max()), float(d.mean())
