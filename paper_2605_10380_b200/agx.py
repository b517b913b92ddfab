"""Thin ctypes binding over ``libagx.so`` (argument marshalling only).

Every function mirrors the C entry point of the same name in ``include/agx.h``; all computation
runs in the CUDA kernels.  Device buffers are ``torch`` tensors (torch is used for allocation and
streams only); host length arrays are numpy ``int32``.  There is no CPU fallback: if the shared
library is missing or fails to load, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional

import numpy as np

AGX_OK = 0
AGX_BF16, AGX_F32 = 0, 1
AGX_DEV_BAD_PAGE, AGX_DEV_WAIT_TIMEOUT, AGX_DEV_BAD_TOKEN = 1, 2, 4
AGX_OPT_EARLY_PREFIX_LOADS, AGX_OPT_WAIT_LIMIT_CYCLES, AGX_OPT_TEST_DROP_STAGE, AGX_OPT_ZERO_COPY = 1, 2, 3, 4
DTYPES = {"bf16": AGX_BF16, "f32": AGX_F32}

_LIB_PATH = Path(__file__).resolve().parent / "lib" / "libagx.so"
_lib = None

EXPORTS = (
    "agx_create", "agx_destroy", "agx_status_string", "agx_last_error", "agx_kv_append",
    "agx_attn_workspace_bytes", "agx_attn_prefixed", "agx_attn_prefixed_append", "agx_accept_workspace_bytes",
    "agx_accept_greedy", "agx_get_status", "agx_last_launch_count",
    "agx_verify_step_host_workspace_bytes", "agx_verify_step_host", "agx_verify_step_host_enqueue",
    "agx_accept_greedy_static", "agx_ngram_lut_bytes", "agx_ngram_workspace_bytes", "agx_ngram_build", "agx_ngram_draft",
    "agx_pw_select_combinations", "agx_pw_longest_prefix", "agx_kv_copy_pages",
    "agx_kv_import_staging_bytes", "agx_kv_import_pages", "agx_set_option",
)


class AgxConfig(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("scale", ctypes.c_float)]


class AgxError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)}) {detail}".rstrip())


def ngram_lut_bytes(max_stream_tokens: int) -> int:
    return int(load().agx_ngram_lut_bytes(int(max_stream_tokens)))


def ngram_workspace_bytes(stream_tokens: int) -> int:
    return int(load().agx_ngram_workspace_bytes(int(stream_tokens)))


def pw_select_combinations(samples, budget: int):
    """samples: list of cluster-id sequences.  Returns (list of selected tuples in order, list of gains)."""
    lib = load()
    n = len(samples)
    max_len = max([len(s) for s in samples] + [1])
    arr = np.full((max(n, 1), max_len), -1, dtype=np.int32)
    for i, s in enumerate(samples):
        arr[i, :len(s)] = np.asarray(s, dtype=np.int32)
    sel = np.full((max(budget, 1), max_len), -1, dtype=np.int32)
    sel_len = np.zeros(max(budget, 1), dtype=np.int32); gains = np.zeros(max(budget, 1), dtype=np.int32)
    cnt = ctypes.c_int32(0)
    st = lib.agx_pw_select_combinations(_ptr(arr), n, max_len, int(budget), _ptr(sel), _ptr(sel_len), _ptr(gains), ctypes.byref(cnt))
    if st != AGX_OK:
        raise AgxError(st, "agx_pw_select_combinations")
    k = int(cnt.value)
    return [tuple(int(c) for c in sel[i, :sel_len[i]]) for i in range(k)], gains[:k].tolist()


def pw_longest_prefix(stored, query):
    """stored: list of cluster-id sequences; query: one sequence.  Returns (index, length)."""
    lib = load()
    max_len = max([len(s) for s in stored] + [1])
    arr = np.full((max(len(stored), 1), max_len), -1, dtype=np.int32)
    lens = np.zeros(max(len(stored), 1), dtype=np.int32)
    for i, s in enumerate(stored):
        arr[i, :len(s)] = np.asarray(s, dtype=np.int32); lens[i] = len(s)
    q = np.asarray(list(query) if len(query) else [0], dtype=np.int32)
    idx, ln = ctypes.c_int32(0), ctypes.c_int32(0)
    st = lib.agx_pw_longest_prefix(_ptr(arr), _ptr(lens), len(stored), max_len, _ptr(q), len(query), ctypes.byref(idx), ctypes.byref(ln))
    if st != AGX_OK:
        raise AgxError(st, "agx_pw_longest_prefix")
    return int(idx.value), int(ln.value)


def lib_path() -> Path:
    return _LIB_PATH


def load() -> ctypes.CDLL:
    """Load the CUDA library; raises if it was not built (run ``python -m paper_2605_10380_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise RuntimeError(f"{_LIB_PATH} is missing: the CUDA library must be built first "
                           "(python -m paper_2605_10380_b200.build); there is no CPU fallback")
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.agx_create.argtypes = [ctypes.POINTER(AgxConfig), ctypes.POINTER(vp)]
    lib.agx_create.restype = i32
    lib.agx_destroy.argtypes = [vp]
    lib.agx_destroy.restype = i32
    lib.agx_status_string.argtypes = [i32]
    lib.agx_status_string.restype = ctypes.c_char_p
    lib.agx_last_error.argtypes = [vp]
    lib.agx_last_error.restype = ctypes.c_char_p
    lib.agx_kv_append.argtypes = [vp, vp, vp, i64, vp, vp, vp, i32, vp, vp, i32, i32, vp]
    lib.agx_kv_append.restype = i32
    lib.agx_attn_workspace_bytes.argtypes = [vp, i32, vp, vp]
    lib.agx_attn_workspace_bytes.restype = i64
    lib.agx_attn_prefixed.argtypes = [vp, vp, vp, vp, i64, vp, i32, vp, vp, i32, vp, vp, vp, ctypes.c_size_t, vp]
    lib.agx_attn_prefixed.restype = i32
    lib.agx_attn_prefixed_append.argtypes = [vp, vp, vp, vp, vp, vp, i64, vp, i32, vp, vp, i32, vp, vp, vp, ctypes.c_size_t, vp]
    lib.agx_attn_prefixed_append.restype = i32
    lib.agx_accept_workspace_bytes.argtypes = [vp, i32, i32]
    lib.agx_accept_workspace_bytes.restype = i64
    lib.agx_accept_greedy.argtypes = [vp, vp, i32, i64, i32, vp, vp, i32, i32, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.agx_accept_greedy.restype = i32
    lib.agx_get_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.agx_get_status.restype = i32
    lib.agx_last_launch_count.argtypes = [vp]
    lib.agx_last_launch_count.restype = i32
    lib.agx_verify_step_host_workspace_bytes.argtypes = [vp, i32, vp, vp, i32, i64, i32]
    lib.agx_verify_step_host_workspace_bytes.restype = i64
    lib.agx_verify_step_host.argtypes = [vp, vp, vp, i64, vp, i32, vp, vp, i32,  # handle .. B
                                         vp, vp, vp, vp, i32, i64, i32, vp,     # host q, k, v, logits .., drafts
                                         vp, vp, vp, vp,                        # host outputs
                                         vp, ctypes.c_size_t, vp]
    lib.agx_verify_step_host.restype = i32
    lib.agx_verify_step_host_enqueue.argtypes = lib.agx_verify_step_host.argtypes
    lib.agx_verify_step_host_enqueue.restype = i32
    lib.agx_accept_greedy_static.argtypes = [vp, i32, i64, i32, vp, vp, i32, i32, vp, vp, vp, vp, vp]
    lib.agx_accept_greedy_static.restype = i32
    lib.agx_ngram_lut_bytes.argtypes = [i32]
    lib.agx_ngram_lut_bytes.restype = i64
    lib.agx_ngram_workspace_bytes.argtypes = [i32]
    lib.agx_ngram_workspace_bytes.restype = i64
    lib.agx_ngram_build.argtypes = [vp, vp, i32, i32, vp, ctypes.c_size_t, vp, ctypes.c_size_t, vp]
    lib.agx_ngram_build.restype = i32
    lib.agx_ngram_draft.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, vp]
    lib.agx_ngram_draft.restype = i32
    lib.agx_pw_select_combinations.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
    lib.agx_pw_select_combinations.restype = i32
    lib.agx_pw_longest_prefix.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp]
    lib.agx_pw_longest_prefix.restype = i32
    lib.agx_kv_copy_pages.argtypes = [vp, vp, vp, i64, vp, vp, i32, vp]
    lib.agx_kv_copy_pages.restype = i32
    lib.agx_kv_import_staging_bytes.argtypes = [vp, i32]
    lib.agx_kv_import_staging_bytes.restype = i64
    lib.agx_kv_import_pages.argtypes = [vp, vp, vp, i64, vp, vp, vp, i32, vp, ctypes.c_size_t, vp]
    lib.agx_kv_import_pages.restype = i32
    lib.agx_set_option.argtypes = [vp, i32, i64]
    lib.agx_set_option.restype = i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().agx_status_string(int(status)).decode()


def _ptr(t) -> Optional[int]:
    """Device pointer of a torch tensor, host pointer of a numpy array, or None."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _h_i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def accept_greedy_static(logits, logits_dtype: str, vocab: int, drafts, cu_q, accept_len, next_token, argmax=None,
                         seq_lens=None, stream=None) -> None:
    """agx_accept_greedy_static: the accept step without handle, workspace or any allocation (for
    callers that may not allocate device memory).  Same tensors as ``Handle.accept_greedy``."""
    B = int(cu_q.shape[0]) - 1
    st = load().agx_accept_greedy_static(_ptr(logits), DTYPES[logits_dtype], int(logits.stride(0)), int(vocab),
                                         _ptr(drafts), _ptr(cu_q), B, int(logits.shape[0]), _ptr(accept_len),
                                         _ptr(next_token), _ptr(argmax), _ptr(seq_lens), _stream_ptr(stream))
    if st != AGX_OK:
        raise AgxError(st, "agx_accept_greedy_static")


class Handle:
    """Owns an ``agx_handle``.  Methods are named after the C calls they forward to."""

    def __init__(self, num_q_heads: int, num_kv_heads: int, head_dim: int, dtype: str = "bf16",
                 scale: float = 0.0, page_size: int = 16):
        self._lib = load()
        self.cfg = AgxConfig(num_q_heads, num_kv_heads, head_dim, page_size, DTYPES[dtype], scale)
        self.dtype = dtype
        self._h = ctypes.c_void_p()
        st = self._lib.agx_create(ctypes.byref(self.cfg), ctypes.byref(self._h))
        if st != AGX_OK:
            raise AgxError(st, "agx_create")

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            self._lib.agx_destroy(self._h)
            self._h = None   # (at interpreter shutdown the ctypes module may already be gone)

    __del__ = close

    def _check(self, st: int, where: str):
        if st != AGX_OK:
            raise AgxError(st, where, self._lib.agx_last_error(self._h).decode())

    # -- agx_set_option
    def set_option(self, option: int, value: int) -> None:
        self._check(self._lib.agx_set_option(self._h, int(option), int(value)), "agx_set_option")

    def last_launch_count(self) -> int:
        return int(self._lib.agx_last_launch_count(self._h))

    # -- agx_kv_append
    def kv_append(self, k_pool, v_pool, k_new, v_new, page_table, prefix_len, cu_q, stream=None):
        B = int(prefix_len.shape[0])
        total_q = int(k_new.shape[0])
        st = self._lib.agx_kv_append(self._h, _ptr(k_pool), _ptr(v_pool), int(k_pool.shape[0]), _ptr(k_new),
                                     _ptr(v_new), _ptr(page_table), int(page_table.shape[1]), _ptr(prefix_len),
                                     _ptr(cu_q), B, total_q, _stream_ptr(stream))
        self._check(st, "agx_kv_append")

    # -- agx_attn_workspace_bytes
    def attn_workspace_bytes(self, h_prefix_len, h_q_len) -> int:
        P, Q = _h_i32(h_prefix_len), _h_i32(h_q_len)
        n = int(self._lib.agx_attn_workspace_bytes(self._h, int(P.shape[0]), _ptr(P), _ptr(Q)))
        if n < 0:
            self._check(n, "agx_attn_workspace_bytes")
        return n

    # -- agx_attn_prefixed
    def attn_prefixed(self, q_block, k_pool, v_pool, page_table, h_prefix_len, h_q_len, out, lse=None,
                      workspace=None, stream=None):
        P, Q = _h_i32(h_prefix_len), _h_i32(h_q_len)
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        st = self._lib.agx_attn_prefixed(self._h, _ptr(q_block), _ptr(k_pool), _ptr(v_pool), int(k_pool.shape[0]),
                                         _ptr(page_table), int(page_table.shape[1]), _ptr(P), _ptr(Q),
                                         int(P.shape[0]), _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes,
                                         _stream_ptr(stream))
        self._check(st, "agx_attn_prefixed")

    # -- agx_attn_prefixed_append
    def attn_prefixed_append(self, q_block, k_new, v_new, k_pool, v_pool, page_table, h_prefix_len, h_q_len, out, lse=None,
                             workspace=None, stream=None):
        P, Q = _h_i32(h_prefix_len), _h_i32(h_q_len)
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        st = self._lib.agx_attn_prefixed_append(self._h, _ptr(q_block), _ptr(k_new), _ptr(v_new), _ptr(k_pool), _ptr(v_pool),
                                                int(k_pool.shape[0]), _ptr(page_table), int(page_table.shape[1]), _ptr(P),
                                                _ptr(Q), int(P.shape[0]), _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes,
                                                _stream_ptr(stream))
        self._check(st, "agx_attn_prefixed_append")

    # -- agx_accept_workspace_bytes
    def accept_workspace_bytes(self, total_q: int, vocab: int) -> int:
        n = int(self._lib.agx_accept_workspace_bytes(self._h, int(total_q), int(vocab)))
        if n < 0:
            self._check(n, "agx_accept_workspace_bytes")
        return n

    # -- agx_accept_greedy
    def accept_greedy(self, logits, logits_dtype: str, vocab: int, drafts, cu_q, accept_len, next_token,
                      argmax=None, seq_lens=None, workspace=None, stream=None):
        B = int(cu_q.shape[0]) - 1
        total_q = int(logits.shape[0])
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        st = self._lib.agx_accept_greedy(self._h, _ptr(logits), DTYPES[logits_dtype], int(logits.stride(0)),
                                         int(vocab), _ptr(drafts), _ptr(cu_q), B, total_q, _ptr(accept_len),
                                         _ptr(next_token), _ptr(argmax), _ptr(seq_lens), _ptr(workspace), ws_bytes,
                                         _stream_ptr(stream))
        self._check(st, "agx_accept_greedy")

    # -- agx_kv_copy_pages (src, dst: device int32 tensors)
    def kv_copy_pages(self, k_pool, v_pool, src, dst, stream=None):
        st = self._lib.agx_kv_copy_pages(self._h, _ptr(k_pool), _ptr(v_pool), int(k_pool.shape[0]), _ptr(src), _ptr(dst),
                                         int(src.numel()), _stream_ptr(stream))
        self._check(st, "agx_kv_copy_pages")

    # -- agx_kv_import_pages (h_k, h_v: pinned host tensors or numpy arrays; dst_pages: device int32; staging: device uint8)
    def kv_import_staging_bytes(self, count: int) -> int:
        return int(self._lib.agx_kv_import_staging_bytes(self._h, int(count)))

    def kv_import_pages(self, k_pool, v_pool, h_k, h_v, dst_pages, staging, stream=None):
        st = self._lib.agx_kv_import_pages(self._h, _ptr(k_pool), _ptr(v_pool), int(k_pool.shape[0]), _ptr(h_k), _ptr(h_v),
                                           _ptr(dst_pages), int(dst_pages.numel()), _ptr(staging),
                                           staging.numel() * staging.element_size(), _stream_ptr(stream))
        self._check(st, "agx_kv_import_pages")

    # -- agx_ngram_build / agx_ngram_draft (device int32 tensors; lut and workspace are uint8 tensors)
    def ngram_build(self, stream_tokens, n: int, lut, workspace, stream=None):
        st = self._lib.agx_ngram_build(self._h, _ptr(stream_tokens), int(stream_tokens.numel()), int(n), _ptr(lut),
                                       lut.numel() * lut.element_size(), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream_ptr(stream))
        self._check(st, "agx_ngram_build")

    def ngram_draft(self, lut, context, fill, k: int, drafts, has_draft, stream=None):
        st = self._lib.agx_ngram_draft(self._h, _ptr(lut), _ptr(context), _ptr(fill), int(has_draft.shape[0]), int(k),
                                       _ptr(drafts), _ptr(has_draft), _stream_ptr(stream))
        self._check(st, "agx_ngram_draft")

    # -- agx_get_status
    def get_status(self, stream=None, raise_on_error: bool = False) -> int:
        v = ctypes.c_int32(0)
        st = self._lib.agx_get_status(self._h, _stream_ptr(stream), ctypes.byref(v))
        if raise_on_error:
            self._check(st, "agx_get_status")
        return int(v.value)

    # -- agx_verify_step_host_workspace_bytes
    def verify_step_host_workspace_bytes(self, h_prefix_len, h_q_len, logits_dtype: str, row_stride: int,
                                         vocab: int) -> int:
        P, Q = _h_i32(h_prefix_len), _h_i32(h_q_len)
        n = int(self._lib.agx_verify_step_host_workspace_bytes(self._h, int(P.shape[0]), _ptr(P), _ptr(Q),
                                                               DTYPES[logits_dtype], int(row_stride), int(vocab)))
        if n < 0:
            self._check(n, "agx_verify_step_host_workspace_bytes")
        return n

    # -- agx_verify_step_host_enqueue with the arguments marshalled once
    def verify_step_host_bind(self, k_pool, v_pool, page_table, h_prefix_len, h_q_len, h_q_block, h_k_new, h_v_new,
                              h_logits, logits_dtype: str, row_stride: int, vocab: int, h_drafts, h_out, h_accept_len,
                              h_next_token, h_seq_lens, workspace, stream=None):
        """Marshal the arguments of ``agx_verify_step_host_enqueue`` once and return a function that makes the
        call (a model that runs the same step over and over pays the conversion of two dozen arguments only
        once).  The returned function keeps every buffer alive; it raises on a non-zero status."""
        P, Q = _h_i32(h_prefix_len), _h_i32(h_q_len)
        keep = (k_pool, v_pool, page_table, P, Q, h_q_block, h_k_new, h_v_new, h_logits, h_drafts, h_out, h_accept_len,
                h_next_token, h_seq_lens, workspace)
        vp = ctypes.c_void_p
        args = (self._h, vp(_ptr(k_pool)), vp(_ptr(v_pool)), ctypes.c_int64(int(k_pool.shape[0])),
                vp(_ptr(page_table)), ctypes.c_int32(int(page_table.shape[1])), vp(_ptr(P)), vp(_ptr(Q)),
                ctypes.c_int32(int(P.shape[0])), vp(_ptr(h_q_block)), vp(_ptr(h_k_new)), vp(_ptr(h_v_new)),
                vp(_ptr(h_logits)), ctypes.c_int32(DTYPES[logits_dtype]), ctypes.c_int64(int(row_stride)), ctypes.c_int32(int(vocab)),
                vp(_ptr(h_drafts)), vp(_ptr(h_out)), vp(_ptr(h_accept_len)), vp(_ptr(h_next_token)),
                vp(_ptr(h_seq_lens)), vp(_ptr(workspace)), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                vp(_stream_ptr(stream)))
        fn = self._lib.agx_verify_step_host_enqueue

        def call(_keep=keep):
            st = fn(*args)
            if st != AGX_OK:
                self._check(st, "agx_verify_step_host_enqueue")
        return call

    # -- agx_verify_step_host (host tensors: pinned torch tensors or numpy arrays)
    def verify_step_host(self, k_pool, v_pool, page_table, h_prefix_len, h_q_len, h_q_block, h_k_new, h_v_new,
                         h_logits, logits_dtype: str, row_stride: int, vocab: int, h_drafts, h_out, h_accept_len,
                         h_next_token, h_seq_lens, workspace, stream=None, enqueue_only: bool = False):
        """agx_verify_step_host, or agx_verify_step_host_enqueue when ``enqueue_only`` (the caller then
        synchronises the stream before reading the host outputs and keeps ``h_prefix_len``/``h_q_len`` and the
        pinned inputs alive until then)."""
        P, Q = _h_i32(h_prefix_len), _h_i32(h_q_len)
        ws_bytes = workspace.numel() * workspace.element_size()
        fn = self._lib.agx_verify_step_host_enqueue if enqueue_only else self._lib.agx_verify_step_host
        st = fn(self._h, _ptr(k_pool), _ptr(v_pool), int(k_pool.shape[0]),
                _ptr(page_table), int(page_table.shape[1]), _ptr(P), _ptr(Q),
                int(P.shape[0]), _ptr(h_q_block), _ptr(h_k_new), _ptr(h_v_new),
                _ptr(h_logits), DTYPES[logits_dtype], int(row_stride), int(vocab),
                _ptr(h_drafts), _ptr(h_out), _ptr(h_accept_len), _ptr(h_next_token),
                _ptr(h_seq_lens), _ptr(workspace), ws_bytes, _stream_ptr(stream))
        self._check(st, "agx_verify_step_host_enqueue" if enqueue_only else "agx_verify_step_host")
