"""CPU oracle (test infrastructure only; never on the product path).

Thin ctypes wrapper over ``agx_oracle.c``: the plain fp64 definition of prefix-cached block
attention (Sec. 2.3, prefix caching), of the verify block (Sec. 2.3, speculative decoding)
and of greedy acceptance.  Only ``tests/``, the smoke check and the benchmark's CPU-baseline
leg import this package.  It imports nothing from the CUDA package.

Arrays use the storage convention of the input generators: ``"bf16"`` arrays are ``uint16``
bit patterns, ``"f32"`` arrays are ``float32``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "agx_oracle.c"
_LIB_PATH = _HERE / "_build" / "libagx_oracle.so"
_lock = threading.Lock()
_lib = None

_DT = {"bf16": 0, "f32": 1}
_NP = {"bf16": np.uint16, "f32": np.float32}


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (OpenMP) if the shared object is missing or stale."""
    if not force and _LIB_PATH.exists() and _LIB_PATH.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB_PATH
    _LIB_PATH.parent.mkdir(parents=True, exist_ok=True)
    tmp = _LIB_PATH.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-fno-fast-math",
           "-ffp-contract=off", str(_SRC), "-o", str(tmp), "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(str(build()))
            lib.oracle_num_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _chk(a: np.ndarray, dtype: str) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != _NP[dtype]:
        raise TypeError(f"expected {_NP[dtype]} storage for dtype {dtype}, got {a.dtype}")
    return a


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def default_scale(d: int) -> float:
    return 1.0 / float(np.sqrt(np.float64(d)))


def attn_contiguous(q_block, K, V, dtype, P, scale=None, select=None):
    """Block attention over contiguous K/V ``[P+q, Hkv, d]``.

    Returns ``(out, lse, psum)``: ``out [q, Hq, d]``, ``lse [q, Hq]``, ``psum [q, Hq]`` (sum of the
    normalised weights, 1 up to rounding), all float64.  ``select=(i_idx, h_idx)`` computes only
    those rows and returns ``[n, d]``, ``[n]``, ``[n]``.
    """
    lib = _load()
    q_block, K, V = _chk(q_block, dtype), _chk(K, dtype), _chk(V, dtype)
    q, hq, d = q_block.shape
    hkv = K.shape[1]
    assert K.shape[0] >= P + q and V.shape == K.shape and hq % hkv == 0
    scale = default_scale(d) if scale is None else float(scale)
    si = sh = None
    n_sel = 0
    if select is not None:
        si, sh = _i32(select[0]), _i32(select[1])
        n_sel = int(si.shape[0])
        out = np.empty((n_sel, d)); lse = np.empty(n_sel); ps = np.empty(n_sel)
    else:
        out = np.empty((q, hq, d)); lse = np.empty((q, hq)); ps = np.empty((q, hq))
    lib.oracle_attn_contiguous(_p(q_block), _p(K), _p(V), _DT[dtype], hq, hkv, d,
                               ctypes.c_int64(P), ctypes.c_int64(q), ctypes.c_double(scale),
                               ctypes.c_int64(n_sel), _p(si), _p(sh), _p(out), _p(lse), _p(ps))
    return out, lse, ps


def attn_paged(q_block, k_pool, v_pool, page_row, dtype, P, scale=None, select=None):
    """Block attention for one sequence whose KV lives in a paged pool ``[pages, Hkv, 16, d]``."""
    lib = _load()
    q_block, k_pool, v_pool = _chk(q_block, dtype), _chk(k_pool, dtype), _chk(v_pool, dtype)
    page_row = _i32(page_row)
    q, hq, d = q_block.shape
    hkv = k_pool.shape[1]
    assert k_pool.shape[2] == 16 and k_pool.shape[3] == d and hq % hkv == 0
    assert page_row.shape[0] * 16 >= P + q
    scale = default_scale(d) if scale is None else float(scale)
    si = sh = None
    n_sel = 0
    if select is not None:
        si, sh = _i32(select[0]), _i32(select[1])
        n_sel = int(si.shape[0])
        out = np.empty((n_sel, d)); lse = np.empty(n_sel); ps = np.empty(n_sel)
    else:
        out = np.empty((q, hq, d)); lse = np.empty((q, hq)); ps = np.empty((q, hq))
    lib.oracle_attn_paged(_p(q_block), _p(k_pool), _p(v_pool), _p(page_row), _DT[dtype], hq, hkv, d,
                          ctypes.c_int64(P), ctypes.c_int64(q), ctypes.c_double(scale),
                          ctypes.c_int64(n_sel), _p(si), _p(sh), _p(out), _p(lse), _p(ps))
    return out, lse, ps


def attn_paged_batch(q_block, k_pool, v_pool, page_table, dtype, prefix_len, q_len, cu_q, scale=None):
    """Ragged batch over a shared paged pool.  Returns ``(out [total_q, Hq, d], lse [total_q, Hq])``."""
    lib = _load()
    q_block, k_pool, v_pool = _chk(q_block, dtype), _chk(k_pool, dtype), _chk(v_pool, dtype)
    page_table = _i32(page_table)
    prefix_len, q_len, cu_q = _i32(prefix_len), _i32(q_len), _i32(cu_q)
    total_q, hq, d = q_block.shape
    hkv = k_pool.shape[1]
    B = prefix_len.shape[0]
    assert int(cu_q[-1]) == total_q
    scale = default_scale(d) if scale is None else float(scale)
    out = np.empty((total_q, hq, d)); lse = np.empty((total_q, hq))
    lib.oracle_attn_paged_batch(_p(q_block), _p(k_pool), _p(v_pool), _p(page_table),
                                ctypes.c_int64(page_table.shape[1]), _DT[dtype], hq, hkv, d, B,
                                _p(prefix_len), _p(q_len), _p(cu_q), ctypes.c_double(scale),
                                _p(out), _p(lse))
    return out, lse


def decode_plain(qv, K, V, dtype, scale=None):
    """Independent single-token decode attention: ``qv [Hq, d]`` against all of ``K, V [L, Hkv, d]``."""
    lib = _load()
    qv, K, V = _chk(qv, dtype), _chk(K, dtype), _chk(V, dtype)
    hq, d = qv.shape
    L, hkv, _ = K.shape
    scale = default_scale(d) if scale is None else float(scale)
    out = np.empty((hq, d))
    lib.oracle_decode_plain(_p(qv), _p(K), _p(V), _DT[dtype], hq, hkv, d, ctypes.c_int64(L),
                            ctypes.c_double(scale), _p(out))
    return out


def kv_append(k_pool, v_pool, k_new, v_new, dtype, page_table, prefix_len, cu_q):
    """In-place append of the block's K/V rows into the pools (storage bits copied)."""
    lib = _load()
    for a in (k_pool, v_pool):
        assert a.flags["C_CONTIGUOUS"] and a.dtype == _NP[dtype]
    k_new, v_new = _chk(k_new, dtype), _chk(v_new, dtype)
    page_table = _i32(page_table)
    prefix_len, cu_q = _i32(prefix_len), _i32(cu_q)
    hkv, d = k_pool.shape[1], k_pool.shape[3]
    lib.oracle_kv_append(_p(k_pool), _p(v_pool), _p(k_new), _p(v_new), _DT[dtype], hkv, d,
                         _p(page_table), ctypes.c_int64(page_table.shape[1]),
                         int(prefix_len.shape[0]), _p(prefix_len), _p(cu_q))


def accept_greedy(logits, dtype, vocab, drafts, cu_q, prefix_len):
    """Greedy acceptance.  Returns ``(argmax [rows], accept_len [B], next_token [B], seq_len [B])``."""
    lib = _load()
    logits = _chk(logits, dtype)
    assert logits.ndim == 2 and logits.shape[1] >= vocab
    drafts, cu_q, prefix_len = _i32(drafts), _i32(cu_q), _i32(prefix_len)
    B = cu_q.shape[0] - 1
    rows = int(cu_q[-1])
    assert logits.shape[0] >= rows and drafts.shape[0] >= rows - B
    am = np.empty(rows, dtype=np.int32)
    al = np.empty(B, dtype=np.int32)
    nt = np.empty(B, dtype=np.int32)
    sl = np.empty(B, dtype=np.int32)
    lib.oracle_accept_greedy(_p(logits), _DT[dtype], ctypes.c_int64(logits.shape[1]), int(vocab),
                             _p(drafts), _p(cu_q), B, _p(prefix_len), _p(am), _p(al), _p(nt), _p(sl))
    return am, al, nt, sl
