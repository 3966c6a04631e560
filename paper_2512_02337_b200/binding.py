"""Thin ctypes binding of libspecpv.so: the same names as include/specpv.h, argument marshalling only.

Every step of the verification path runs in the library's CUDA kernels; this module converts
torch tensors to raw pointers and raises :class:`SpecPVError` on a non-zero status.  There is no
fallback: if the shared library is missing, importing the symbols fails loudly.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, c_float, c_int, c_int32, c_size_t, c_void_p
from dataclasses import dataclass
from pathlib import Path

import numpy as np
import torch

LIB_PATH = Path(__file__).resolve().parent / "lib" / "libspecpv.so"

STATUS_NAMES = ["OK", "INVALID_ARG", "SHAPE", "BUDGET", "CAPACITY", "BAD_TREE", "BAD_BLOCK_TABLE",
                "UNSUPPORTED", "CUDA", "TIMEOUT"]
DTYPE_F32, DTYPE_BF16 = 0, 1
REDUCE_MEAN, REDUCE_MAX, REDUCE_LAST = 0, 1, 2
MODE_FULL, MODE_PARTIAL, MODE_REFRESH = 0, 1, 2

EXPORTS = [
    "specpv_status_string", "specpv_workspace_bytes", "specpv_kernel_launches", "specpv_poll_status", "specpv_build_tree_mask",
    "specpv_select_mode", "specpv_update_block_summaries", "specpv_score_blocks",
    "specpv_select_partial_kv", "specpv_refresh_partial", "specpv_verify_partial",
    "specpv_verify_full", "specpv_verify_host", "specpv_commit_accepted", "specpv_verify_partial_static",
    "specpv_rope_table", "specpv_qkv_rope", "specpv_o_proj", "specpv_verify_full_offloaded",
]


SELFTEST_EXPORTS = ["specpv_selftest_wait_timeout"]  # include/specpv_selftest.h
SELFTEST_WHERE = 99


class SpecPVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: SPECPV_ERR_{name}")


class Config(ctypes.Structure):
    """Mirror of ``specpv_config``."""
    _fields_ = [("n_layers", c_int32), ("n_q_heads", c_int32), ("n_kv_heads", c_int32),
                ("head_dim", c_int32), ("block_tokens", c_int32), ("dtype", c_int32),
                ("sink_blocks", c_int32), ("local_blocks", c_int32), ("budget_blocks", c_int32),
                ("buffer_tokens", c_int32), ("reduce", c_int32), ("score_mode", c_int32),
                ("softmax_scale", c_float), ("out_f32", c_int32), ("select_shared", c_int32)]


class PagedKV(ctypes.Structure):
    """Mirror of ``specpv_paged_kv``."""
    _fields_ = [("k_pool", c_void_p), ("v_pool", c_void_p), ("block_table", c_void_p),
                ("seq_lens", c_void_p), ("batch", c_int32), ("max_blocks", c_int32),
                ("n_pages", c_int32), ("max_seq_len", c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libspecpv.so (raises if it has not been built -- there is no other code path)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2512_02337_b200.build` "
                              "(the CUDA library is the only implementation)")
        _lib = ctypes.CDLL(str(LIB_PATH))
        _lib.specpv_status_string.restype = ctypes.c_char_p
        _lib.specpv_workspace_bytes.restype = c_size_t
        _lib.specpv_workspace_bytes.argtypes = [POINTER(Config), c_int, c_int, c_int, c_int]
        _lib.specpv_kernel_launches.restype = ctypes.c_uint64
        for name in EXPORTS[3:] + SELFTEST_EXPORTS:
            getattr(_lib, name).restype = c_int
    return _lib


def _ptr(t) -> c_void_p:
    if t is None:
        return c_void_p(0)
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensors passed to the C ABI must be contiguous"
        return c_void_p(t.data_ptr())
    if isinstance(t, np.ndarray):
        assert t.flags.c_contiguous
        return c_void_p(t.ctypes.data)
    raise TypeError(type(t))


def _stream(stream) -> c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(status: int, where: str):
    if status != 0:
        raise SpecPVError(status, where)


def make_config(n_layers, n_q_heads, n_kv_heads, head_dim, block_tokens, dtype, sink_blocks, local_blocks,
                budget_blocks, buffer_tokens, reduce=REDUCE_MEAN, score_mode=0, softmax_scale=0.0, out_f32=0, select_shared=0) -> Config:
    code = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16, "fp32": DTYPE_F32, "bf16": DTYPE_BF16}.get(dtype, dtype)
    return Config(n_layers, n_q_heads, n_kv_heads, head_dim, block_tokens, code, sink_blocks, local_blocks,
                  budget_blocks, buffer_tokens, reduce, score_mode, softmax_scale, out_f32, select_shared)


@dataclass
class Cache:
    """A paged KV cache (full or partial) as torch tensors plus its C descriptor."""
    k_pool: torch.Tensor       # [n_layers][n_pages][Hkv][bs][d]
    v_pool: torch.Tensor
    block_table: torch.Tensor  # [batch][max_blocks] int32
    seq_lens: torch.Tensor     # [batch] int32
    max_seq_len: int

    def desc(self) -> PagedKV:
        batch, max_blocks = self.block_table.shape
        return PagedKV(self.k_pool.data_ptr(), self.v_pool.data_ptr(), self.block_table.data_ptr(),
                       self.seq_lens.data_ptr(), batch, max_blocks, self.k_pool.shape[1], int(self.max_seq_len))


def specpv_status_string(status: int) -> str:
    return lib().specpv_status_string(c_int(status)).decode()


def specpv_workspace_bytes(cfg: Config, n_layers_per_call: int, max_batch: int, max_seq_len: int, M_max: int) -> int:
    return int(lib().specpv_workspace_bytes(ctypes.byref(cfg), n_layers_per_call, max_batch, max_seq_len, M_max))


def specpv_kernel_launches() -> int:
    return int(lib().specpv_kernel_launches())


def new_workspace(cfg: Config, n_layers_per_call: int, max_batch: int, max_seq_len: int, M_max: int,
                  device="cuda") -> torch.Tensor:
    """Allocate and zero a workspace with torch (device memory is the caller's)."""
    n = specpv_workspace_bytes(cfg, n_layers_per_call, max_batch, max_seq_len, M_max)
    if n == 0:
        raise SpecPVError(1, "specpv_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


def specpv_poll_status(workspace: torch.Tensor, stream=None):
    info = (c_int32 * 4)()
    st = lib().specpv_poll_status(_ptr(workspace), _stream(stream), info)
    return st, list(info)


def specpv_build_tree_mask(parents, n_chain: int = 0, row_words: int | None = None) -> np.ndarray:
    parents = np.ascontiguousarray(parents, dtype=np.int32)
    M = parents.shape[0] + n_chain
    if row_words is None:
        row_words = (M + 63) // 64
    mask = np.zeros((M, row_words), dtype=np.uint64)
    _check(lib().specpv_build_tree_mask(_ptr(parents), parents.shape[0], n_chain, _ptr(mask), row_words),
           "specpv_build_tree_mask")
    return mask


def specpv_select_mode(ctx_len, budget_tokens, n_partially_verified, n_candidates, buffer_tokens,
                       partial_initialised) -> int:
    return lib().specpv_select_mode(ctx_len, budget_tokens, n_partially_verified, n_candidates, buffer_tokens,
                                    int(bool(partial_initialised)))


def specpv_update_block_summaries(cfg, layer0, n_layers, kv: Cache, tok_begin, max_blocks_touched, kmax, kmin,
                                  workspace, stream=None):
    d = kv.desc()
    _check(lib().specpv_update_block_summaries(ctypes.byref(cfg), layer0, n_layers, ctypes.byref(d), _ptr(tok_begin),
                                               max_blocks_touched, _ptr(kmax), _ptr(kmin), _ptr(workspace),
                                               c_size_t(workspace.numel()), _stream(stream)),
           "specpv_update_block_summaries")


def specpv_score_blocks(cfg, layer0, n_layers, q, q_lens, M_max, last_query, kmax, kmin, kv: Cache, scores,
                        workspace, stream=None):
    d = kv.desc()
    _check(lib().specpv_score_blocks(ctypes.byref(cfg), layer0, n_layers, _ptr(q), _ptr(q_lens), M_max,
                                     _ptr(last_query), _ptr(kmax), _ptr(kmin), ctypes.byref(d), _ptr(scores),
                                     _ptr(workspace), c_size_t(workspace.numel()), _stream(stream)),
           "specpv_score_blocks")


def specpv_select_partial_kv(cfg, n_layers, scores, seq_lens, batch, max_blocks, idx, count, workspace, stream=None):
    _check(lib().specpv_select_partial_kv(ctypes.byref(cfg), n_layers, _ptr(scores), _ptr(seq_lens), batch,
                                          max_blocks, _ptr(idx), _ptr(count), _ptr(workspace),
                                          c_size_t(workspace.numel()), _stream(stream)),
           "specpv_select_partial_kv")


def specpv_refresh_partial(cfg, full: Cache, idx, count, partial: Cache, partial_lens, workspace, stream=None):
    fd, pd = full.desc(), partial.desc()
    _check(lib().specpv_refresh_partial(ctypes.byref(cfg), ctypes.byref(fd), _ptr(idx), _ptr(count), ctypes.byref(pd),
                                        _ptr(partial_lens), _ptr(workspace), c_size_t(workspace.numel()),
                                        _stream(stream)),
           "specpv_refresh_partial")


def _verify(fn_name, cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max, kv: Cache, out, lse,
            workspace, stream):
    d = kv.desc()
    _check(getattr(lib(), fn_name)(ctypes.byref(cfg), layer0, n_layers, _ptr(q), _ptr(k_new), _ptr(v_new),
                                   _ptr(tree_mask), _ptr(q_lens), M_max, ctypes.byref(d), _ptr(out), _ptr(lse),
                                   _ptr(workspace), c_size_t(workspace.numel()), _stream(stream)), fn_name)


def specpv_verify_partial(cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max, partial: Cache, out,
                          lse, workspace, stream=None):
    _verify("specpv_verify_partial", cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max, partial,
            out, lse, workspace, stream)


STATIC_SCRATCH_BYTES = 16 << 20
WORKSPACE_HEAD_BYTES = 256 << 10  # SPECPV_WORKSPACE_HEAD_BYTES: status word and arrival counters, zero between calls


def specpv_verify_partial_static(cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max, partial: Cache,
                                 out, lse, device_status=None, stream=None):
    """specpv_verify_partial without a workspace: the scratch is a fixed array inside the library, so the
    call allocates nothing (for callers whose device memory is all spoken for).  ``device_status`` is an
    optional int32 device tensor of 5 words that receives the call's device-side status."""
    d = partial.desc()
    _check(lib().specpv_verify_partial_static(ctypes.byref(cfg), layer0, n_layers, _ptr(q), _ptr(k_new), _ptr(v_new),
                                              _ptr(tree_mask), _ptr(q_lens), M_max, ctypes.byref(d), _ptr(out),
                                              _ptr(lse), _ptr(device_status), _stream(stream)),
           "specpv_verify_partial_static")


def specpv_selftest_wait_timeout(workspace, limit_us: int, observed_ns=None, stream=None):
    """Self-test (include/specpv_selftest.h): a bounded barrier wait that runs out after ``limit_us`` microseconds and
    records SPECPV_ERR_TIMEOUT in the workspace's status word.  ``observed_ns``: optional uint64/int64 device tensor."""
    _check(lib().specpv_selftest_wait_timeout(_ptr(workspace), c_size_t(workspace.numel() * workspace.element_size()),
                                              int(limit_us), _ptr(observed_ns), _stream(stream)),
           "specpv_selftest_wait_timeout")


def specpv_verify_full(cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max, full: Cache, out, lse,
                       workspace, stream=None):
    _verify("specpv_verify_full", cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max, full, out,
            lse, workspace, stream)


def specpv_verify_host(cfg, mode, layer0, n_layers, q_host, k_new_host, v_new_host, tree_mask_host, M_max,
                       kv: Cache, out_host, lse_host, workspace, stream=None):
    d = kv.desc()
    _check(lib().specpv_verify_host(ctypes.byref(cfg), mode, layer0, n_layers, _ptr(q_host), _ptr(k_new_host),
                                    _ptr(v_new_host), _ptr(tree_mask_host), M_max, ctypes.byref(d), _ptr(out_host),
                                    _ptr(lse_host), _ptr(workspace), c_size_t(workspace.numel()), _stream(stream)),
           "specpv_verify_host")


def specpv_commit_accepted(cfg, layer0, n_layers, k_new, v_new, M_max, accepted, n_accepted, A_max, dst: Cache,
                           kmax, kmin, workspace, stream=None):
    d = dst.desc()
    _check(lib().specpv_commit_accepted(ctypes.byref(cfg), layer0, n_layers, _ptr(k_new), _ptr(v_new), M_max,
                                        _ptr(accepted), _ptr(n_accepted), A_max, ctypes.byref(d), _ptr(kmax),
                                        _ptr(kmin), _ptr(workspace), c_size_t(workspace.numel()), _stream(stream)),
           "specpv_commit_accepted")


# ---- the linear maps either side of the attention ---------------------------------------------------------------
def specpv_rope_table(cfg, tree_mask, q_lens, base_pos, batch, M_max, rope_theta, cos_sin, stream=None):
    _check(lib().specpv_rope_table(ctypes.byref(cfg), _ptr(tree_mask), _ptr(q_lens), _ptr(base_pos), batch, M_max,
                                   ctypes.c_double(rope_theta), _ptr(cos_sin), _stream(stream)),
           "specpv_rope_table")


def specpv_qkv_rope(cfg, layer0, n_layers, x, hidden, w_qkv, cos_sin, batch, M_max, q, k_new, v_new, workspace,
                    stream=None):
    _check(lib().specpv_qkv_rope(ctypes.byref(cfg), layer0, n_layers, _ptr(x), hidden, _ptr(w_qkv), _ptr(cos_sin),
                                 batch, M_max, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(workspace),
                                 c_size_t(workspace.numel()), _stream(stream)),
           "specpv_qkv_rope")


def specpv_o_proj(cfg, layer0, n_layers, attn, w_o, hidden, residual, batch, M_max, y, workspace, stream=None):
    _check(lib().specpv_o_proj(ctypes.byref(cfg), layer0, n_layers, _ptr(attn), _ptr(w_o), hidden, _ptr(residual),
                               batch, M_max, _ptr(y), _ptr(workspace), c_size_t(workspace.numel()), _stream(stream)),
           "specpv_o_proj")


# ---- full KV cache in host memory -------------------------------------------------------------------------------
class OffloadedKV(ctypes.Structure):
    """Mirror of ``specpv_offloaded_kv``."""
    _fields_ = [("k_host", c_void_p), ("v_host", c_void_p), ("k_stage", c_void_p), ("v_stage", c_void_p),
                ("block_table", c_void_p), ("seq_lens", c_void_p), ("batch", c_int32), ("max_blocks", c_int32),
                ("n_pages", c_int32), ("max_seq_len", c_int32)]


@dataclass
class OffloadedCache:
    """A full cache in pinned host memory plus the two device layer slots a full verification stages through."""
    k_host: torch.Tensor       # pinned host, [n_layers][n_pages][Hkv][bs][d]
    v_host: torch.Tensor
    k_stage: torch.Tensor      # device, [2][n_pages][Hkv][bs][d]
    v_stage: torch.Tensor
    block_table: torch.Tensor  # device
    seq_lens: torch.Tensor     # device
    max_seq_len: int

    def desc(self) -> OffloadedKV:
        assert self.k_host.is_pinned() and self.v_host.is_pinned(), "the offloaded pools must be page-locked"
        batch, max_blocks = self.block_table.shape
        return OffloadedKV(self.k_host.data_ptr(), self.v_host.data_ptr(), self.k_stage.data_ptr(),
                           self.v_stage.data_ptr(), self.block_table.data_ptr(), self.seq_lens.data_ptr(), batch,
                           max_blocks, self.k_host.shape[1], int(self.max_seq_len))

    def as_cache(self) -> Cache:
        """The host pools as an ordinary cache descriptor (commit and gather address them in place)."""
        return Cache(self.k_host, self.v_host, self.block_table, self.seq_lens, self.max_seq_len)


def specpv_verify_full_offloaded(cfg, layer0, n_layers, q, k_new, v_new, tree_mask, q_lens, M_max,
                                 full: OffloadedCache, out, lse, workspace, stream=None, copy_stream=None):
    d = full.desc()
    _check(lib().specpv_verify_full_offloaded(ctypes.byref(cfg), layer0, n_layers, _ptr(q), _ptr(k_new), _ptr(v_new),
                                              _ptr(tree_mask), _ptr(q_lens), M_max, ctypes.byref(d), _ptr(out),
                                              _ptr(lse), _ptr(workspace), c_size_t(workspace.numel()),
                                              _stream(stream), _stream(copy_stream)),
           "specpv_verify_full_offloaded")
