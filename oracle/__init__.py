"""float64 CPU oracle of the SpecPV verification hot path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline / reference legs may import
this package.  The CUDA library and its Python binding never do.  The arithmetic lives in
``specpv_oracle.c`` (plain C, double accumulation, written from the paper's Section 3.2-3.3,
Eq. 1-3 and Algorithm 1); this module only builds it with gcc and marshals numpy arrays.

Array conventions: float32 data is ``np.float32``; bfloat16 data is carried as raw
``np.uint16`` bit patterns (numpy has no bfloat16).  ``dtype`` code: 0 = float32, 1 = bfloat16.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "specpv_oracle.c"
_LIB = _HERE / "libspecpv_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (OpenMP).  Building the checker is not using it."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-fvisibility=hidden", "-std=c11",
             "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.oracle_tree_mask.restype = ctypes.c_int
        _lib.oracle_select.restype = ctypes.c_int
        _lib.oracle_gather.restype = ctypes.c_int
        _lib.oracle_commit.restype = ctypes.c_int
        _lib.oracle_select_mode.restype = ctypes.c_int
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_block_summaries.restype = None
        _lib.oracle_block_scores.restype = None
        _lib.oracle_block_scores_mode.restype = None
        _lib.oracle_tree_attention.restype = None
        _lib.oracle_step_positions.restype = ctypes.c_int
        _lib.oracle_linear.restype = None
        _lib.oracle_rope.restype = None
        _lib.oracle_qkv_rope.restype = None
    return _lib


def _p(a):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def _code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError(f"oracle buffers are float32 or uint16 (bf16 bits), got {a.dtype}")


def _c(a, dtype=None):
    a = np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return _load().oracle_num_threads()


def widen(a: np.ndarray) -> np.ndarray:
    """Exact float64 value of a float32 / bf16-bits array (a format conversion, no arithmetic)."""
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def tree_mask(parents, n_chain: int = 0) -> np.ndarray:
    """Ancestor-or-self mask [M][W] uint64 of a chain of n_chain tokens followed by the tree."""
    parents = _c(parents, np.int32)
    n_tree = parents.shape[0]
    M = n_tree + n_chain
    W = (M + 63) // 64
    mask = np.zeros((M, W), dtype=np.uint64)
    rc = _load().oracle_tree_mask(_p(parents), n_tree, n_chain, _p(mask))
    if rc != 0:
        raise ValueError("parents[] is not a tree in topological order")
    return mask


def block_summaries(k_pool, block_table, seq_len: int):
    """Eq. 1 for one layer and one sequence.  k_pool [n_pages][Hkv][bs][d] -> (kmax, kmin) [Hkv][nb][d] f64."""
    k_pool = _c(k_pool)
    _, Hkv, bs, d = k_pool.shape
    block_table = _c(block_table, np.int32)
    nb = (seq_len + bs - 1) // bs
    kmax = np.empty((Hkv, nb, d), dtype=np.float64)
    kmin = np.empty((Hkv, nb, d), dtype=np.float64)
    _load().oracle_block_summaries(_p(k_pool), _code(k_pool), Hkv, bs, d, _p(block_table), seq_len,
                                   _p(kmax), _p(kmin))
    return kmax, kmin


def block_scores(q, kmax, kmin, Hkv: int, reduce: int = 0, last_query: int = 0, score_mode: int = 0) -> np.ndarray:
    """Eq. 2-3.  q [M][Hq][d]; kmax/kmin [Hkv][nb][d] f64 -> scores [Hkv][nb] f64.

    score_mode 0 is Eq. 2 as printed; 1 is the channel-wise form sum_c max(q_c Kmax_c, q_c Kmin_c)."""
    q = _c(q)
    M, Hq, d = q.shape
    kmax = _c(kmax, np.float64)
    kmin = _c(kmin, np.float64)
    nb = kmax.shape[1]
    scores = np.empty((Hkv, nb), dtype=np.float64)
    _load().oracle_block_scores_mode(_p(q), _code(q), M, Hq, Hkv, d, _p(kmax), _p(kmin), nb,
                                     reduce, last_query, score_mode, _p(scores))
    return scores


def select(scores, sink_blocks: int, local_blocks: int, budget_blocks: int) -> np.ndarray:
    """Retained block indices (ascending) for one (layer, sequence, KV head)."""
    scores = _c(scores, np.float64)
    nb = scores.shape[0]
    idx = np.empty(max(nb, budget_blocks), dtype=np.int32)
    n = _load().oracle_select(_p(scores), nb, sink_blocks, local_blocks, budget_blocks, _p(idx))
    return idx[:n].copy()


def head_shared_scores(scores) -> np.ndarray:
    """Scores that head-shared selection ranks on: the mean over the KV heads of one layer and sequence.

    scores [Hkv][nb] -> [nb] float64: the plain mean, in double precision; the selection itself is :func:`select`
    on the result."""
    return np.asarray(scores, dtype=np.float64).mean(axis=0)


def gather(k_pool, v_pool, block_table, seq_len: int, idx, pk_pool, pv_pool, first_page: int) -> int:
    """Copy the selected blocks of every KV head into the partial pool; returns the partial length."""
    k_pool, v_pool = _c(k_pool), _c(v_pool)
    _, Hkv, bs, d = k_pool.shape
    block_table = _c(block_table, np.int32)
    idx = _c(idx, np.int32)
    assert idx.ndim == 2 and idx.shape[0] == Hkv
    assert pk_pool.flags.c_contiguous and pv_pool.flags.c_contiguous
    return _load().oracle_gather(_p(k_pool), _p(v_pool), _code(k_pool), Hkv, bs, d, _p(block_table),
                                 seq_len, _p(idx), idx.shape[1], idx.shape[1], _p(pk_pool), _p(pv_pool),
                                 first_page)


def tree_attention(q, knew, vnew, mask, k_pool, v_pool, block_table, seq_len: int,
                   scale: float | None = None, want_probs: bool = False):
    """Tree-masked GQA attention of one layer and one sequence -> (out [M][Hq][d], lse [M][Hq]) f64."""
    q, knew, vnew = _c(q), _c(knew), _c(vnew)
    k_pool, v_pool = _c(k_pool), _c(v_pool)
    M, Hq, d = q.shape
    _, Hkv, bs, _ = k_pool.shape
    assert knew.shape == (M, Hkv, d) and vnew.shape == (M, Hkv, d)
    mask = _c(mask, np.uint64)
    assert mask.shape == (M, (M + 63) // 64)
    block_table = _c(block_table, np.int32)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.empty((M, Hq, d), dtype=np.float64)
    lse = np.empty((M, Hq), dtype=np.float64)
    probs = np.empty((M, Hq, seq_len + M), dtype=np.float64) if want_probs else None
    _load().oracle_tree_attention(_p(q), _p(knew), _p(vnew), _code(q), M, Hq, Hkv, d, _p(mask),
                                  _p(k_pool), _p(v_pool), bs, _p(block_table), seq_len,
                                  ctypes.c_double(scale), _p(out), _p(lse), _p(probs))
    return (out, lse, probs) if want_probs else (out, lse)


def commit(knew, vnew, accepted, k_pool, v_pool, block_table, seq_len: int) -> int:
    """Append rows `accepted` of Knew/Vnew to the cache in place; returns the new length."""
    knew, vnew = _c(knew), _c(vnew)
    _, Hkv, bs, d = k_pool.shape
    accepted = _c(accepted, np.int32)
    block_table = _c(block_table, np.int32)
    assert k_pool.flags.c_contiguous and v_pool.flags.c_contiguous
    return _load().oracle_commit(_p(knew), _p(vnew), _code(knew), Hkv, bs, d, _p(accepted),
                                 accepted.shape[0], _p(k_pool), _p(v_pool), _p(block_table), seq_len)


FULL, PARTIAL, REFRESH = 0, 1, 2


def select_mode(ctx_len: int, budget_tokens: int, n_partially_verified: int, n_candidates: int,
                buffer_tokens: int, partial_initialised: bool) -> int:
    return _load().oracle_select_mode(ctx_len, budget_tokens, n_partially_verified, n_candidates,
                                      buffer_tokens, int(bool(partial_initialised)))


# ---- the linear maps either side of the attention (Algorithm 1 "TreeDecode") ------------------------------------
def step_positions(parents, n_chain: int = 0, base: int = 0) -> np.ndarray:
    """Sequence positions of a step's rows: chain rows base.., tree node at base + n_chain + depth."""
    parents = _c(parents, np.int32)
    pos = np.empty(parents.shape[0] + n_chain, dtype=np.int32)
    if _load().oracle_step_positions(_p(parents), parents.shape[0], n_chain, base, _p(pos)) != 0:
        raise ValueError("parents[] is not a tree in topological order")
    return pos


def linear(x, w, residual=None) -> np.ndarray:
    """y = x w^T (+ residual).  x [T][n_in], w [n_out][n_in] (float32 or bf16 bits) -> [T][n_out] f64."""
    x, w = _c(x), _c(w)
    assert _code(x) == _code(w) and x.shape[1] == w.shape[1]
    if residual is not None:
        residual = _c(residual)
        assert _code(residual) == _code(x) and residual.shape == (x.shape[0], w.shape[0])
    y = np.empty((x.shape[0], w.shape[0]), dtype=np.float64)
    _load().oracle_linear(_p(x), _p(w), _code(x), x.shape[0], x.shape[1], w.shape[0], _p(residual), _p(y))
    return y


def rope(a, pos, theta: float) -> np.ndarray:
    """Rotary embedding (half-split pairing) of a [T][H][d] float64 array at positions pos [T]; returns a copy."""
    a = np.array(a, dtype=np.float64, order="C")
    T, H, d = a.shape
    pos = _c(pos, np.int32)
    assert pos.shape == (T,)
    _load().oracle_rope(_p(a), T, H, d, _p(pos), ctypes.c_double(theta))
    return a


def qkv_rope(x, w_qkv, Hq: int, Hkv: int, d: int, pos, theta: float):
    """x [T][hidden], w_qkv [(Hq+2Hkv)d][hidden] -> (q [T][Hq][d], k [T][Hkv][d], v [T][Hkv][d]) f64."""
    x, w_qkv = _c(x), _c(w_qkv)
    T, hidden = x.shape
    assert w_qkv.shape == ((Hq + 2 * Hkv) * d, hidden) and _code(x) == _code(w_qkv)
    pos = _c(pos, np.int32)
    q = np.empty((T, Hq, d), dtype=np.float64)
    k = np.empty((T, Hkv, d), dtype=np.float64)
    v = np.empty((T, Hkv, d), dtype=np.float64)
    _load().oracle_qkv_rope(_p(x), _p(w_qkv), _code(x), T, hidden, Hq, Hkv, d, _p(pos), ctypes.c_double(theta),
                            _p(q), _p(k), _p(v))
    return q, k, v
