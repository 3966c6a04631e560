"""Test-side helpers: run the CPU oracle on slices of a workload and compare with the CUDA library."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl

# tolerances of the floating-point outputs: max-abs and relative RMS, per storage dtype.
# bfloat16 runs are checked on the float32 output (cfg.out_f32 = 1): the workloads' outputs reach
# |o| >= 8, where rounding the result to bfloat16 alone costs up to 0.031; the bfloat16 output is
# checked separately to be exactly the rounded float32 output (same_as_rounded).
TOL = {"fp32": (1e-5, 1e-5), "bf16": (2e-2, 5e-3)}


def same_as_rounded(out_bf16: torch.Tensor, out_f32: torch.Tensor):
    """The bfloat16 output must be the float32 output rounded to nearest-even, bit for bit."""
    assert out_bf16.dtype == torch.bfloat16 and out_f32.dtype == torch.float32
    assert torch.equal(out_bf16, out_f32.to(torch.bfloat16))


def config_for(w: wl.Workload, **over) -> B.Config:
    c = w.cfg
    sink, local = wl.sink_local_blocks(c["bs"])
    kw = dict(n_layers=c["n_layers"], n_q_heads=c["Hq"], n_kv_heads=c["Hkv"], head_dim=c["d"],
              block_tokens=c["bs"], dtype=c["dtype"], sink_blocks=sink, local_blocks=local,
              budget_blocks=c["budget_blocks"], buffer_tokens=c["buffer_tokens"], out_f32=1)
    kw.update(over)
    return B.make_config(**kw)


def full_cache(w: wl.Workload) -> B.Cache:
    return B.Cache(w.k_pool, w.v_pool, w.block_table, w.seq_lens, int(max(w.cfg["ctx"])))


def device_masks(parents: np.ndarray, M_max: int, n_chain: int = 0, device="cuda") -> torch.Tensor:
    """[batch][M_max][W] uint64 masks built by the library's host routine, as an int64 device tensor."""
    W = (M_max + 63) // 64
    rows = []
    for p in parents:
        m = B.specpv_build_tree_mask(p, n_chain, W)
        pad = np.zeros((M_max, W), dtype=np.uint64)
        pad[: m.shape[0]] = m
        rows.append(pad)
    return torch.from_numpy(np.stack(rows).view(np.int64)).to(device)


def compare(got: np.ndarray, want: np.ndarray, dtype: str, what: str = ""):
    """max-abs and relative-RMS check of a floating-point output against the oracle (float64)."""
    max_abs_tol, rel_rms_tol = TOL[dtype]
    got = got.astype(np.float64)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    err = np.abs(got - want)
    rel_rms = np.sqrt((err ** 2).mean()) / max(np.sqrt((want ** 2).mean()), 1e-30)
    assert err.max() <= max_abs_tol, f"{what}: max-abs {err.max():.3e} > {max_abs_tol}"
    assert rel_rms <= rel_rms_tol, f"{what}: rel-RMS {rel_rms:.3e} > {rel_rms_tol}"
    return err.max(), rel_rms


def widen_t(t: torch.Tensor) -> np.ndarray:
    return oracle.widen(wl.to_numpy(t))


def oracle_attention_rows(q, k_new, v_new, parents, n_chain, rows, k_pool, v_pool, table, seq_len, scale=None):
    """Oracle attention for a subset of step rows closed under ancestry.

    ``rows`` are indices into the step's tokens (chain tokens first, then tree nodes); the closure
    under parents is taken, the sub-tree renumbered, and the oracle run on it.  Because a token only
    sees its ancestors among the step's tokens, its output equals its output in the full step.
    Returns (closed_rows, out [n][Hq][d], lse [n][Hq])."""
    n_tree = len(parents)
    M = n_chain + n_tree
    comb = np.concatenate([np.arange(-1, n_chain - 1), np.where(np.asarray(parents) < 0, n_chain - 1,
                                                                np.asarray(parents) + n_chain)]).astype(np.int64)
    keep = set()
    for r in rows:
        a = int(r)
        while a >= 0 and a not in keep:
            keep.add(a)
            a = int(comb[a])
    closed = np.array(sorted(keep), dtype=np.int64)
    renum = {int(r): i for i, r in enumerate(closed)}
    sub_parents = np.array([renum[int(comb[r])] if comb[r] >= 0 else -1 for r in closed], dtype=np.int32)
    assert M >= len(closed)
    mask = oracle.tree_mask(sub_parents)
    out, lse = oracle.tree_attention(q[closed], k_new[closed], v_new[closed], mask, k_pool, v_pool, table,
                                     seq_len, scale)
    return closed, out, lse


def sync_status(ws: torch.Tensor, expect: int = 0):
    st, info = B.specpv_poll_status(ws)
    assert st == expect, f"device status {st} ({B.specpv_status_string(st)}), info {info}"


def check_shared_selection(idx_row: np.ndarray, scores: np.ndarray, sink: int, local: int, budget: int, what: str = ""):
    """Head-shared selection: the kernel ranks blocks on a float32 mean over the KV heads; the oracle's definition is
    the float64 mean.  Where the two rankings can differ only through float32 rounding (means of the last kept and the
    first dropped block closer than that rounding), any choice among the tied blocks is correct; everywhere else the
    list must be the oracle's.  scores [Hkv][nb] are the kernel's own float32 scores."""
    Hkv, nb = scores.shape
    mean = oracle.head_shared_scores(scores)
    want = oracle.select(mean, sink, local, budget)
    got = np.asarray(idx_row)
    if np.array_equal(got, want):
        return
    # rounding of a float32 sum of Hkv terms and one multiplication
    eps = (Hkv + 1) * 2.0 ** -23 * float(np.abs(scores).max())
    assert len(got) == len(want), f"{what}: {len(got)} blocks kept, oracle keeps {len(want)}"
    assert np.all(np.diff(got) > 0), f"{what}: block list not ascending"
    must = set(range(min(sink, nb))) | set(range(max(nb - local, 0), nb))
    assert must <= set(got.tolist()), f"{what}: sink or local blocks missing"
    kept = sorted(set(got.tolist()) - must)
    dropped = sorted(set(range(sink, nb - local)) - set(kept))
    if kept and dropped:
        assert mean[kept].min() >= mean[dropped].max() - eps, f"{what}: a dropped block outranks a kept one beyond rounding"
    # what differs from the oracle's list lies within rounding of the cut
    diff = sorted(set(got.tolist()) ^ set(want.tolist()))
    cut = mean[sorted(set(want.tolist()) - must)].min() if set(want.tolist()) - must else 0.0
    assert np.all(np.abs(mean[diff] - cut) <= eps), f"{what}: lists differ away from the cut"
