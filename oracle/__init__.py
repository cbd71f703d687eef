"""CPU oracle for one batched tree-verification step -- TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``reader_oracle.c`` (plain C, fp64).  Only tests, the
smoke check and the CPU-baseline leg of the benchmark may import this module;
the product package never does, and this module never imports the product's
CUDA binding.  Arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import POINTER, c_double, c_float, c_int, c_int32, c_int64, c_uint8, c_uint16, c_void_p

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "reader_oracle.c")
_LIB = os.path.join(_HERE, "libreader_oracle.so")

OK, BAD_TREE, CAPACITY, BAD_PAGE = 0, 2, 3, 8


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p16, p32, pf, pd = POINTER(c_uint16), POINTER(c_int32), POINTER(c_float), POINTER(c_double)
        lib.oracle_num_threads.restype = c_int
        lib.oracle_set_num_threads.argtypes = [c_int]
        lib.oracle_tree_is_valid.argtypes = [p32, c_int]
        lib.oracle_tree_is_valid.restype = c_int
        lib.oracle_ancestor_matrix.argtypes = [p32, c_int, POINTER(c_uint8)]
        lib.oracle_levels.argtypes = [p32, c_int, p32]
        lib.oracle_verify_attn.argtypes = [p16, p16, p16, p16, p16, c_int, c_int, c_int, c_int,
                                           p32, c_int, p32, p32, c_int, c_int, c_int, c_double,
                                           pd, c_void_p, c_void_p, c_int64, p32]
        lib.oracle_argmax.argtypes = [pf, c_int64, c_int64, p32]
        lib.oracle_kv_rearrange.argtypes = [p16, p16, c_int, c_int, c_int, c_int, POINTER(c_uint8), p32]
        lib.oracle_verify_attn_padded.argtypes = [p16, p16, p16, p16, p16, c_int, c_int, c_int, POINTER(c_uint8), c_int,
                                                  p32, c_int, c_int, c_int, c_double, pd, c_void_p, p32]
        lib.oracle_padded_append.argtypes = [p16, p16, c_int, c_int, c_int, c_int, POINTER(c_uint8), p32, p16, p16,
                                             c_int, p32, p32, c_int, p32]
        lib.oracle_sample_targets.argtypes = [pf, p32, pf, c_int, c_int, c_int64, c_double, c_int64, c_float, p32]
        lib.oracle_accept.argtypes = [p32, p32, p32, c_int, c_int, c_int, p32, p32, p32, p32]
        lib.oracle_kv_commit.argtypes = [p16, p16, c_int, c_int, c_int, c_int, p32, c_int, p32, c_int,
                                         p16, p16, c_int, c_int, p32, p32, c_int, c_int, p32, p32]
        _lib = lib
    return _lib


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _ptr(a, ctype):
    return a.ctypes.data_as(POINTER(ctype))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def tree_is_valid(parent) -> bool:
    parent = _c(parent, np.int32)
    return bool(_load().oracle_tree_is_valid(_ptr(parent, c_int32), parent.shape[-1]))


def ancestor_matrix(parent) -> np.ndarray:
    """M[i, j] = 1 iff node i is node j or one of its ancestors (Sec. 3.2 mask, made reflexive)."""
    parent = _c(parent, np.int32)
    T = parent.shape[0]
    M = np.zeros((T, T), dtype=np.uint8)
    _load().oracle_ancestor_matrix(_ptr(parent, c_int32), T, _ptr(M, c_uint8))
    return M


def levels(parent) -> np.ndarray:
    parent = _c(parent, np.int32)
    out = np.zeros(parent.shape[0], dtype=np.int32)
    _load().oracle_levels(_ptr(parent, c_int32), parent.shape[0], _ptr(out, c_int32))
    return out


def verify_attn(q, k_tree, v_tree, k_pool, v_pool, page_table, seq_lens, parent, scale,
                want_lse: bool = False, want_probs: bool = False):
    """Sec. 3.2 tree attention in fp64.

    q [B,T,Hq,D], k_tree/v_tree [B,T,Hkv,D], k_pool/v_pool [num_pages,Hkv,P,D] (all uint16 bf16
    bits), page_table [B,max_pages] i32, seq_lens [B] i32, parent [B,T] i32.
    Returns dict(out=f64 [B,T,Hq,D], status=i32 [B], lse=..., probs=[B,T,Hq,maxL+T]).
    """
    q, k_tree, v_tree = _c(q, np.uint16), _c(k_tree, np.uint16), _c(v_tree, np.uint16)
    k_pool, v_pool = _c(k_pool, np.uint16), _c(v_pool, np.uint16)
    page_table, seq_lens, parent = _c(page_table, np.int32), _c(seq_lens, np.int32), _c(parent, np.int32)
    B, T, Hq, D = q.shape
    num_pages, Hkv, P, _ = k_pool.shape
    assert k_tree.shape == (B, T, Hkv, D) and v_tree.shape == k_tree.shape and v_pool.shape == k_pool.shape
    assert page_table.shape[0] == B and seq_lens.shape == (B,) and parent.shape == (B, T)
    out = np.zeros((B, T, Hq, D), dtype=np.float64)
    status = np.zeros(B, dtype=np.int32)
    lse = np.zeros((B, T, Hq), dtype=np.float64) if want_lse else None
    stride = int(max(int(seq_lens.max(initial=0)), 0) + T)
    probs = np.zeros((B, T, Hq, stride), dtype=np.float64) if want_probs else None
    _load().oracle_verify_attn(
        _ptr(q, c_uint16), _ptr(k_tree, c_uint16), _ptr(v_tree, c_uint16),
        _ptr(k_pool, c_uint16), _ptr(v_pool, c_uint16), num_pages, P, Hkv, D,
        _ptr(page_table, c_int32), page_table.shape[1], _ptr(seq_lens, c_int32),
        _ptr(parent, c_int32), B, T, Hq, float(scale), _ptr(out, c_double),
        lse.ctypes.data if lse is not None else None,
        probs.ctypes.data if probs is not None else None, stride, _ptr(status, c_int32))
    res = {"out": out, "status": status}
    if want_lse:
        res["lse"] = lse
    if want_probs:
        res["probs"] = probs
    return res


def argmax(logits) -> np.ndarray:
    """First index of each row's maximum; logits f32 [..., V] -> i32 [...]."""
    logits = _c(logits, np.float32)
    V = logits.shape[-1]
    rows = logits.size // V if V else 0
    out = np.zeros(rows, dtype=np.int32)
    _load().oracle_argmax(_ptr(logits, c_float), rows, V, _ptr(out, c_int32))
    return out.reshape(logits.shape[:-1])


def kv_rearrange(k, v, valid):
    """Algorithm 4 on a padded batch cache k, v [B, Hkv, cap, D] (uint16 bf16 bits) with a validity
    mask [B, cap]; works on copies.  Returns dict(k, v, valid, lengths)."""
    k, v = _c(k, np.uint16).copy(), _c(v, np.uint16).copy()
    valid = _c(valid, np.uint8).copy()
    B, Hkv, cap, D = k.shape
    assert v.shape == k.shape and valid.shape == (B, cap)
    lengths = np.zeros(B, dtype=np.int32)
    _load().oracle_kv_rearrange(_ptr(k, c_uint16), _ptr(v, c_uint16), B, Hkv, cap, D, _ptr(valid, c_uint8),
                                _ptr(lengths, c_int32))
    return {"k": k, "v": v, "valid": valid, "lengths": lengths}


def verify_attn_padded(q, k_tree, v_tree, k, v, valid, extent: int, parent, scale, want_lse: bool = False):
    """Sec. 3.2 attention over the padded batch cache of Sec. 4.3: k, v [B, Hkv, cap, D] (uint16 bf16
    bits), valid [B, cap] u8, common length `extent`.  Returns dict(out, status[, lse])."""
    q, k_tree, v_tree = _c(q, np.uint16), _c(k_tree, np.uint16), _c(v_tree, np.uint16)
    k, v, valid, parent = _c(k, np.uint16), _c(v, np.uint16), _c(valid, np.uint8), _c(parent, np.int32)
    B, T, Hq, D = q.shape
    _, Hkv, cap, _ = k.shape
    assert k.shape == (B, Hkv, cap, D) and v.shape == k.shape and valid.shape == (B, cap)
    assert k_tree.shape == (B, T, Hkv, D) and v_tree.shape == k_tree.shape and parent.shape == (B, T)
    out = np.zeros((B, T, Hq, D), dtype=np.float64)
    lse = np.zeros((B, T, Hq), dtype=np.float64) if want_lse else None
    status = np.zeros(B, dtype=np.int32)
    _load().oracle_verify_attn_padded(
        _ptr(q, c_uint16), _ptr(k_tree, c_uint16), _ptr(v_tree, c_uint16), _ptr(k, c_uint16), _ptr(v, c_uint16),
        cap, Hkv, D, _ptr(valid, c_uint8), int(extent), _ptr(parent, c_int32), B, T, Hq, float(scale),
        _ptr(out, c_double), lse.ctypes.data if lse is not None else None, _ptr(status, c_int32))
    res = {"out": out, "status": status}
    if want_lse:
        res["lse"] = lse
    return res


def padded_append(k, v, valid, extent: int, k_tree, v_tree, path, n_acc):
    """One step's growth of the padded batch cache (Sec. 4.3), on copies: the accepted rows behind the
    common length, zero rows up to the batch's longest span.  Returns dict(k, v, valid, extent, status)."""
    k, v, valid = _c(k, np.uint16).copy(), _c(v, np.uint16).copy(), _c(valid, np.uint8).copy()
    k_tree, v_tree = _c(k_tree, np.uint16), _c(v_tree, np.uint16)
    path, n_acc = _c(path, np.int32), _c(n_acc, np.int32)
    B, Hkv, cap, D = k.shape
    T = k_tree.shape[1]
    ext = np.array([extent], dtype=np.int32)
    status = np.zeros(B, dtype=np.int32)
    _load().oracle_padded_append(_ptr(k, c_uint16), _ptr(v, c_uint16), B, Hkv, cap, D, _ptr(valid, c_uint8),
                                 _ptr(ext, c_int32), _ptr(k_tree, c_uint16), _ptr(v_tree, c_uint16), T,
                                 _ptr(path, c_int32), _ptr(n_acc, c_int32), path.shape[1], _ptr(status, c_int32))
    return {"k": k, "v": v, "valid": valid, "extent": int(ext[0]), "status": status}


def sample_targets(logits, parent, uniforms, temperature: float, top_k: int = 0, top_p: float = 1.0) -> np.ndarray:
    """Appendix C, randomized policy: per-node target id x* = F(P, U) by temperature inverse-CDF
    sampling; uniforms f32 [B, T], entry level-1 serves all nodes of that tree level.  top_k > 0 keeps
    only the logits that are at least the top_k-th largest of their row (ties kept); top_p < 1 then keeps
    the smallest set of highest logits whose weight reaches that share (ties kept)."""
    logits, parent, uniforms = _c(logits, np.float32), _c(parent, np.int32), _c(uniforms, np.float32)
    B, T = parent.shape
    V = logits.shape[-1]
    assert logits.shape == (B, T, V) and uniforms.shape == (B, T)
    out = np.zeros((B, T), dtype=np.int32)
    _load().oracle_sample_targets(_ptr(logits, c_float), _ptr(parent, c_int32), _ptr(uniforms, c_float), B, T, V,
                                  float(temperature), int(top_k), float(top_p), _ptr(out, c_int32))
    return out


def accept(parent, node_tokens, target_ids, max_path: int):
    """Longest consistent root path (Algorithm 5) -> dict(path, n_acc, bonus, status)."""
    parent, tok, tgt = _c(parent, np.int32), _c(node_tokens, np.int32), _c(target_ids, np.int32)
    B, T = parent.shape
    path = np.zeros((B, max_path), dtype=np.int32)
    n_acc = np.zeros(B, dtype=np.int32)
    bonus = np.zeros(B, dtype=np.int32)
    status = np.zeros(B, dtype=np.int32)
    _load().oracle_accept(_ptr(parent, c_int32), _ptr(tok, c_int32), _ptr(tgt, c_int32), B, T, max_path,
                          _ptr(path, c_int32), _ptr(n_acc, c_int32), _ptr(bonus, c_int32), _ptr(status, c_int32))
    return {"path": path, "n_acc": n_acc, "bonus": bonus, "status": status}


def kv_commit(k_pool, v_pool, page_table, seq_lens, shared_prefix_len, k_tree, v_tree, path, n_acc,
              update_seq_lens: bool = True):
    """Append the accepted nodes' K/V behind each sequence (Sec. 4.3, Algorithm 4), on copies.

    Returns dict(k_pool, v_pool, seq_lens, slots, status); the inputs are not modified.
    """
    k_pool, v_pool = _c(k_pool, np.uint16).copy(), _c(v_pool, np.uint16).copy()
    page_table, seq_lens = _c(page_table, np.int32), _c(seq_lens, np.int32).copy()
    k_tree, v_tree = _c(k_tree, np.uint16), _c(v_tree, np.uint16)
    path, n_acc = _c(path, np.int32), _c(n_acc, np.int32)
    num_pages, Hkv, P, D = k_pool.shape
    B, T = k_tree.shape[:2]
    max_path = path.shape[1]
    slots = np.zeros((B, max_path), dtype=np.int32)
    status = np.zeros(B, dtype=np.int32)
    _load().oracle_kv_commit(_ptr(k_pool, c_uint16), _ptr(v_pool, c_uint16), num_pages, P, Hkv, D,
                             _ptr(page_table, c_int32), page_table.shape[1], _ptr(seq_lens, c_int32),
                             int(shared_prefix_len), _ptr(k_tree, c_uint16), _ptr(v_tree, c_uint16), B, T,
                             _ptr(path, c_int32), _ptr(n_acc, c_int32), max_path, int(bool(update_seq_lens)),
                             _ptr(slots, c_int32), _ptr(status, c_int32))
    return {"k_pool": k_pool, "v_pool": v_pool, "seq_lens": seq_lens, "slots": slots, "status": status}
