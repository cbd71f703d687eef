"""ctypes binding of ``libreader_verify.so``: argument marshalling only.

Every step of the verification path runs in the library's CUDA kernels.  PyTorch is used for
device memory and streams; tensors are passed as raw device pointers.  bf16 tensors are
``torch.bfloat16``.  There is no CPU fallback: if the library is missing or no CUDA device is
present, calls raise.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_float, c_int32, c_size_t, c_void_p
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libreader_verify.so")

(OK, ERR_INVALID_ARG, ERR_BAD_TREE, ERR_CAPACITY, ERR_WORKSPACE, ERR_UNSUPPORTED, ERR_TIMEOUT, ERR_CUDA, ERR_BAD_PAGE,
 ERR_TOO_LARGE) = range(10)
NOALLOC_MAX_ROWS = 4096

EXPORTS = ("reader_create", "reader_destroy", "reader_status_string", "reader_set_attn_kernel", "reader_set_partition",
           "reader_set_timing_events", "reader_set_accept_timing_events",
           "reader_workspace_bytes", "reader_tree_encode", "reader_verify_attn", "reader_accept",
           "reader_kv_commit", "reader_accept_noalloc", "reader_sample_targets", "reader_kv_rearrange", "reader_kv_commit_layers",
           "reader_accept_commit", "reader_verify_prepare", "reader_verify_attn_prepared",
           "reader_padded_workspace_bytes", "reader_verify_attn_padded", "reader_padded_append", "reader_padded_rearrange")


class ReaderError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


class _KvCache(Structure):
    _fields_ = [("k_pool", c_void_p), ("v_pool", c_void_p), ("num_pages", c_int32), ("page_size", c_int32),
                ("n_kv_heads", c_int32), ("head_dim", c_int32), ("page_table", c_void_p),
                ("max_pages_per_seq", c_int32), ("seq_lens", c_void_p), ("shared_prefix_len", c_int32)]


class _PaddedCache(Structure):
    _fields_ = [("k", c_void_p), ("v", c_void_p), ("valid", c_void_p), ("extent", c_void_p), ("capacity", c_int32),
                ("n_kv_heads", c_int32), ("head_dim", c_int32)]


class _Tree(Structure):
    _fields_ = [("batch", c_int32), ("n_nodes", c_int32), ("parent", c_void_p), ("anc_mask", c_void_p)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads the shared library (no CUDA call is made by loading it)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2508_09072_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    lib.reader_create.argtypes = [POINTER(c_void_p), c_int32]
    lib.reader_create.restype = c_int32
    lib.reader_destroy.argtypes = [c_void_p]
    lib.reader_destroy.restype = None
    lib.reader_status_string.argtypes = [c_int32]
    lib.reader_status_string.restype = ctypes.c_char_p
    lib.reader_set_attn_kernel.argtypes = [c_void_p, c_int32]
    lib.reader_set_attn_kernel.restype = c_int32
    lib.reader_set_partition.argtypes = [c_void_p, c_int32]
    lib.reader_set_partition.restype = c_int32
    lib.reader_set_timing_events.argtypes = [c_void_p, c_void_p, c_void_p]
    lib.reader_set_timing_events.restype = c_int32
    lib.reader_set_accept_timing_events.argtypes = [c_void_p, c_void_p, c_void_p]
    lib.reader_set_accept_timing_events.restype = c_int32
    lib.reader_workspace_bytes.argtypes = [c_void_p, c_int32, c_int32, c_int32, c_int32, c_int32]
    lib.reader_workspace_bytes.restype = c_size_t
    lib.reader_tree_encode.argtypes = [c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.reader_tree_encode.restype = c_int32
    lib.reader_verify_attn.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, POINTER(_KvCache),
                                       POINTER(_Tree), c_float, c_void_p, c_void_p, c_void_p, c_size_t,
                                       c_void_p, c_void_p]
    lib.reader_verify_attn.restype = c_int32
    lib.reader_accept.argtypes = [c_void_p, POINTER(_Tree), c_void_p, c_void_p, c_int32, c_void_p, c_int32,
                                  c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.reader_accept.restype = c_int32
    lib.reader_accept_noalloc.argtypes = [c_void_p, POINTER(_Tree), c_void_p, c_void_p, c_int32, c_void_p, c_int32,
                                          c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.reader_accept_noalloc.restype = c_int32
    lib.reader_sample_targets.argtypes = [c_void_p, POINTER(_Tree), c_void_p, c_int32, c_void_p, c_float, c_int32, c_float,
                                          c_void_p, c_void_p]
    lib.reader_sample_targets.restype = c_int32
    lib.reader_kv_commit_layers.argtypes = [c_void_p, POINTER(_KvCache), POINTER(c_void_p), POINTER(c_void_p), c_int32,
                                            c_int32, c_int32, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p,
                                            c_void_p]
    lib.reader_kv_commit_layers.restype = c_int32
    lib.reader_kv_rearrange.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_int32, c_void_p,
                                        c_void_p, c_void_p]
    lib.reader_kv_rearrange.restype = c_int32
    lib.reader_verify_prepare.argtypes = [c_void_p, POINTER(_KvCache), POINTER(_Tree), c_int32, c_void_p, c_size_t, c_void_p,
                                          c_void_p]
    lib.reader_verify_prepare.restype = c_int32
    lib.reader_verify_attn_prepared.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, POINTER(_KvCache),
                                                POINTER(_Tree), c_float, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.reader_verify_attn_prepared.restype = c_int32
    lib.reader_accept_commit.argtypes = [c_void_p, POINTER(_Tree), c_void_p, c_void_p, c_int32, c_void_p, c_int32,
                                         POINTER(_KvCache), c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p,
                                         c_void_p, c_void_p, c_size_t, c_void_p, c_void_p, c_void_p]
    lib.reader_accept_commit.restype = c_int32
    lib.reader_padded_workspace_bytes.argtypes = [c_void_p, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32]
    lib.reader_padded_workspace_bytes.restype = c_size_t
    lib.reader_verify_attn_padded.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, POINTER(_PaddedCache),
                                              POINTER(_Tree), c_float, c_void_p, c_void_p, c_void_p, c_size_t,
                                              c_void_p, c_void_p]
    lib.reader_verify_attn_padded.restype = c_int32
    lib.reader_padded_append.argtypes = [c_void_p, POINTER(_PaddedCache), c_void_p, c_void_p, c_int32, c_int32, c_void_p,
                                         c_void_p, c_int32, c_void_p, c_void_p]
    lib.reader_padded_append.restype = c_int32
    lib.reader_padded_rearrange.argtypes = [c_void_p, POINTER(_PaddedCache), c_int32, c_void_p, c_void_p]
    lib.reader_padded_rearrange.restype = c_int32
    lib.reader_kv_commit.argtypes = [c_void_p, POINTER(_KvCache), c_void_p, c_void_p, c_int32, c_int32, c_void_p,
                                     c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p]
    lib.reader_kv_commit.restype = c_int32
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().reader_status_string(int(code)).decode()


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else c_void_p(t.data_ptr())


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: need a contiguous CUDA tensor of dtype {dtype}")
    return t


def _stream() -> c_void_p:
    return c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class KvCache:
    """One layer's paged cache; tensors live on the device and are owned by the caller."""
    k_pool: torch.Tensor      # bf16 [num_pages, Hkv, page_size, D]
    v_pool: torch.Tensor
    page_table: torch.Tensor  # i32 [B, max_pages]
    seq_lens: torch.Tensor    # i32 [B]
    shared_prefix_len: int = 0

    def _c(self) -> _KvCache:
        _dev(self.k_pool, torch.bfloat16, "k_pool"); _dev(self.v_pool, torch.bfloat16, "v_pool")
        _dev(self.page_table, torch.int32, "page_table"); _dev(self.seq_lens, torch.int32, "seq_lens")
        n, h, p, d = self.k_pool.shape
        return _KvCache(self.k_pool.data_ptr(), self.v_pool.data_ptr(), n, p, h, d, self.page_table.data_ptr(),
                        self.page_table.shape[1], self.seq_lens.data_ptr(), int(self.shared_prefix_len))


@dataclass
class PaddedCache:
    """The padded batch cache of Sec. 4.3; tensors live on the device and are owned by the caller."""
    k: torch.Tensor        # bf16 [B, Hkv, capacity, D]
    v: torch.Tensor
    valid: torch.Tensor    # u8 [B, capacity]
    extent: torch.Tensor   # i32 [1]: the common length

    def _c(self) -> _PaddedCache:
        _dev(self.k, torch.bfloat16, "k"); _dev(self.v, torch.bfloat16, "v")
        _dev(self.valid, torch.uint8, "valid"); _dev(self.extent, torch.int32, "extent")
        B, Hkv, cap, D = self.k.shape
        if self.v.shape != self.k.shape or self.valid.shape != (B, cap) or self.extent.numel() != 1:
            raise ValueError("padded cache: k, v [B, Hkv, cap, D], valid [B, cap], extent [1]")
        return _PaddedCache(self.k.data_ptr(), self.v.data_ptr(), self.valid.data_ptr(), self.extent.data_ptr(), cap, Hkv, D)


class Reader:
    """Handle on the library for one CUDA device (wraps reader_create / reader_destroy)."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2508_09072_b200 needs a CUDA device; there is no CPU fallback")
        self.lib = load_library()
        self.device = int(device)
        torch.cuda.set_device(self.device)
        torch.zeros(1, device=f"cuda:{self.device}")   # make sure the context exists
        h = c_void_p()
        st = self.lib.reader_create(ctypes.byref(h), self.device)
        if st != OK:
            raise ReaderError(st, "reader_create")
        self._h = h
        self._ws: Optional[torch.Tensor] = None

    def close(self):
        if getattr(self, "_h", None):
            self.lib.reader_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- helpers
    def set_attn_kernel(self, which: int) -> None:
        st = self.lib.reader_set_attn_kernel(self._h, int(which))
        if st != OK:
            raise ReaderError(st, "reader_set_attn_kernel")

    def set_partition(self, which: int) -> None:
        """0 automatic, 1 equal ranges, 2 aligned partition whenever a prefix is shared."""
        st = self.lib.reader_set_partition(self._h, int(which))
        if st != OK:
            raise ReaderError(st, "reader_set_partition")

    def set_timing_events(self, start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]) -> None:
        """Events (created with enable_timing=True and already recorded once, so that their handles
        exist) that reader_verify_attn records around its main kernel; None, None turns it off."""
        a = None if start is None else c_void_p(start.cuda_event)
        b = None if stop is None else c_void_p(stop.cuda_event)
        st = self.lib.reader_set_timing_events(self._h, a, b)
        if st != OK:
            raise ReaderError(st, "reader_set_timing_events")

    def set_accept_timing_events(self, start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]) -> None:
        """Events that reader_accept (with logits) records around its argmax kernel; None, None turns it off."""
        a = None if start is None else c_void_p(start.cuda_event)
        b = None if stop is None else c_void_p(stop.cuda_event)
        st = self.lib.reader_set_accept_timing_events(self._h, a, b)
        if st != OK:
            raise ReaderError(st, "reader_set_accept_timing_events")

    def workspace_bytes(self, max_batch: int, max_nodes: int, n_q_heads: int, n_kv_heads: int, head_dim: int) -> int:
        return int(self.lib.reader_workspace_bytes(self._h, max_batch, max_nodes, n_q_heads, n_kv_heads, head_dim))

    def workspace(self, max_batch: int, max_nodes: int, n_q_heads: int, n_kv_heads: int, head_dim: int) -> torch.Tensor:
        """A cached device buffer large enough for the given limits (torch allocation)."""
        need = self.workspace_bytes(max_batch, max_nodes, n_q_heads, n_kv_heads, head_dim)
        if need == 0:
            raise ReaderError(ERR_INVALID_ARG, "reader_workspace_bytes")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}")
        return self._ws

    # ---- the calls
    def tree_encode(self, parent: torch.Tensor, anc_mask: Optional[torch.Tensor] = None,
                    level: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None):
        _dev(parent, torch.int32, "parent")
        B, T = parent.shape
        dev = parent.device
        anc_mask = anc_mask if anc_mask is not None else torch.empty((B, T, 2), dtype=torch.int64, device=dev)
        level = level if level is not None else torch.empty((B, T), dtype=torch.int32, device=dev)
        status = status if status is not None else torch.empty(B, dtype=torch.int32, device=dev)
        st = self.lib.reader_tree_encode(self._h, _ptr(parent), B, T, _ptr(anc_mask), _ptr(level), _ptr(status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_tree_encode")
        return anc_mask, level, status

    def verify_attn(self, q: torch.Tensor, k_tree: torch.Tensor, v_tree: torch.Tensor, cache: KvCache,
                    parent: torch.Tensor, scale: float, anc_mask: Optional[torch.Tensor] = None,
                    out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                    status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
        _dev(q, torch.bfloat16, "q"); _dev(k_tree, torch.bfloat16, "k_tree"); _dev(v_tree, torch.bfloat16, "v_tree")
        _dev(parent, torch.int32, "parent")
        B, T, Hq, D = q.shape
        Hkv = k_tree.shape[2]
        out = out if out is not None else torch.empty_like(q)
        status = status if status is not None else torch.empty(B, dtype=torch.int32, device=q.device)
        ws = workspace if workspace is not None else self.workspace(max(B, 1), T, Hq, Hkv, D)
        tree = _Tree(B, T, parent.data_ptr(), None if anc_mask is None else anc_mask.data_ptr())
        c = cache._c()
        st = self.lib.reader_verify_attn(self._h, _ptr(q), Hq, _ptr(k_tree), _ptr(v_tree), ctypes.byref(c),
                                         ctypes.byref(tree), float(scale), _ptr(out), _ptr(lse), _ptr(ws),
                                         ws.numel(), _ptr(status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_verify_attn")
        return out, status

    def verify_prepare(self, cache: KvCache, parent: torch.Tensor, n_q_heads: int, anc_mask: Optional[torch.Tensor] = None,
                       status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
        """reader_verify_prepare: the per-step part of verify_attn (checks, masks, work partition), once for
        all layers.  Returns (status, workspace); pass both tensors' owners on to verify_attn_prepared."""
        _dev(parent, torch.int32, "parent")
        B, T = parent.shape
        c = cache._c()
        status = status if status is not None else torch.empty(B, dtype=torch.int32, device=parent.device)
        ws = workspace if workspace is not None else self.workspace(max(B, 1), T, n_q_heads, c.n_kv_heads, c.head_dim)
        tree = _Tree(B, T, parent.data_ptr(), None if anc_mask is None else anc_mask.data_ptr())
        st = self.lib.reader_verify_prepare(self._h, ctypes.byref(c), ctypes.byref(tree), int(n_q_heads), _ptr(ws), ws.numel(),
                                            _ptr(status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_verify_prepare")
        return status, ws

    def verify_attn_prepared(self, q: torch.Tensor, k_tree: torch.Tensor, v_tree: torch.Tensor, cache: KvCache,
                             parent: torch.Tensor, scale: float, workspace: torch.Tensor,
                             anc_mask: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                             lse: Optional[torch.Tensor] = None):
        """reader_verify_attn_prepared: one layer's attention and combine on the schedule verify_prepare left
        in `workspace`."""
        _dev(q, torch.bfloat16, "q"); _dev(k_tree, torch.bfloat16, "k_tree"); _dev(v_tree, torch.bfloat16, "v_tree")
        B, T, Hq, D = q.shape
        out = out if out is not None else torch.empty_like(q)
        tree = _Tree(B, T, parent.data_ptr(), None if anc_mask is None else anc_mask.data_ptr())
        c = cache._c()
        st = self.lib.reader_verify_attn_prepared(self._h, _ptr(q), Hq, _ptr(k_tree), _ptr(v_tree), ctypes.byref(c),
                                                  ctypes.byref(tree), float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
                                                  workspace.numel(), _stream())
        if st != OK:
            raise ReaderError(st, "reader_verify_attn_prepared")
        return out

    def verify_attn_padded(self, q: torch.Tensor, k_tree: torch.Tensor, v_tree: torch.Tensor, cache: PaddedCache,
                           parent: torch.Tensor, scale: float, anc_mask: Optional[torch.Tensor] = None,
                           out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                           status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
        """reader_verify_attn_padded: the same attention over the padded batch cache of Sec. 4.3."""
        _dev(q, torch.bfloat16, "q"); _dev(k_tree, torch.bfloat16, "k_tree"); _dev(v_tree, torch.bfloat16, "v_tree")
        _dev(parent, torch.int32, "parent")
        B, T, Hq, D = q.shape
        Hkv = k_tree.shape[2]
        c = cache._c()
        out = out if out is not None else torch.empty_like(q)
        status = status if status is not None else torch.empty(B, dtype=torch.int32, device=q.device)
        if workspace is None:
            need = int(self.lib.reader_padded_workspace_bytes(self._h, max(B, 1), T, Hq, Hkv, D, c.capacity))
            if need == 0:
                raise ReaderError(ERR_INVALID_ARG, "reader_padded_workspace_bytes")
            if self._ws is None or self._ws.numel() < need:
                self._ws = torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}")
            workspace = self._ws
        tree = _Tree(B, T, parent.data_ptr(), None if anc_mask is None else anc_mask.data_ptr())
        st = self.lib.reader_verify_attn_padded(self._h, _ptr(q), Hq, _ptr(k_tree), _ptr(v_tree), ctypes.byref(c),
                                                ctypes.byref(tree), float(scale), _ptr(out), _ptr(lse), _ptr(workspace),
                                                workspace.numel(), _ptr(status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_verify_attn_padded")
        return out, status

    def padded_append(self, cache: PaddedCache, k_tree: torch.Tensor, v_tree: torch.Tensor, path: torch.Tensor,
                      n_acc: torch.Tensor, status: Optional[torch.Tensor] = None) -> torch.Tensor:
        """reader_padded_append: one step's accepted rows behind the common length, zero rows for the rest."""
        _dev(k_tree, torch.bfloat16, "k_tree"); _dev(v_tree, torch.bfloat16, "v_tree")
        _dev(path, torch.int32, "path"); _dev(n_acc, torch.int32, "n_acc")
        B, T = k_tree.shape[:2]
        c = cache._c()
        status = status if status is not None else torch.empty(B, dtype=torch.int32, device=k_tree.device)
        st = self.lib.reader_padded_append(self._h, ctypes.byref(c), _ptr(k_tree), _ptr(v_tree), B, T, _ptr(path), _ptr(n_acc),
                                           path.shape[1] if path.dim() == 2 else 1, _ptr(status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_padded_append")
        return status

    def padded_rearrange(self, cache: PaddedCache, lengths: Optional[torch.Tensor] = None) -> torch.Tensor:
        """reader_padded_rearrange: Algorithm 4 on the whole cache; the common length becomes the longest row."""
        c = cache._c()
        B = cache.k.shape[0]
        if lengths is None:
            lengths = torch.empty(B, dtype=torch.int32, device=cache.k.device)
        st = self.lib.reader_padded_rearrange(self._h, ctypes.byref(c), B, _ptr(lengths), _stream())
        if st != OK:
            raise ReaderError(st, "reader_padded_rearrange")
        return lengths

    def accept(self, parent: torch.Tensor, node_tokens: torch.Tensor, max_path: int,
               logits: Optional[torch.Tensor] = None, target_ids: Optional[torch.Tensor] = None,
               workspace: Optional[torch.Tensor] = None, outs=None):
        _dev(parent, torch.int32, "parent"); _dev(node_tokens, torch.int32, "node_tokens")
        B, T = parent.shape
        dev = parent.device
        vocab = 0
        if logits is not None:
            _dev(logits, torch.float32, "logits")
            vocab = logits.shape[-1]
            if target_ids is None:
                target_ids = torch.empty((B, T), dtype=torch.int32, device=dev)
        elif target_ids is None:
            raise TypeError("accept: give logits or target_ids")
        _dev(target_ids, torch.int32, "target_ids")
        if outs is None:
            outs = (torch.empty((B, max_path), dtype=torch.int32, device=dev),
                    torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev),
                    torch.empty(B, dtype=torch.int32, device=dev))
        path, n_acc, bonus, status = outs
        ws = workspace if workspace is not None else self.workspace(max(B, 1), T, 1, 1, 64)
        tree = _Tree(B, T, parent.data_ptr(), None)
        st = self.lib.reader_accept(self._h, ctypes.byref(tree), _ptr(node_tokens), _ptr(logits), vocab,
                                    _ptr(target_ids), int(max_path), _ptr(path), _ptr(n_acc), _ptr(bonus),
                                    _ptr(ws), ws.numel(), _ptr(status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_accept")
        return {"path": path, "n_acc": n_acc, "bonus": bonus, "status": status, "target_ids": target_ids}

    def accept_commit(self, parent: torch.Tensor, node_tokens: torch.Tensor, max_path: int, cache: KvCache,
                      k_tree: torch.Tensor, v_tree: torch.Tensor, logits: Optional[torch.Tensor] = None,
                      target_ids: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, outs=None,
                      slots: Optional[torch.Tensor] = None, commit_status: Optional[torch.Tensor] = None,
                      update_seq_lens: bool = True):
        """reader_accept_commit: accept() and kv_commit() with the walk and the commit in one launch.
        Returns a dict: path, n_acc, bonus, status, target_ids, slots, commit_status."""
        _dev(parent, torch.int32, "parent"); _dev(node_tokens, torch.int32, "node_tokens")
        _dev(k_tree, torch.bfloat16, "k_tree"); _dev(v_tree, torch.bfloat16, "v_tree")
        B, T = parent.shape
        dev = parent.device
        vocab = 0
        if logits is not None:
            _dev(logits, torch.float32, "logits")
            vocab = logits.shape[-1]
            if target_ids is None:
                target_ids = torch.empty((B, T), dtype=torch.int32, device=dev)
        elif target_ids is None:
            raise TypeError("accept_commit: give logits or target_ids")
        _dev(target_ids, torch.int32, "target_ids")
        if outs is None:
            outs = (torch.empty((B, max_path), dtype=torch.int32, device=dev),
                    torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev),
                    torch.empty(B, dtype=torch.int32, device=dev))
        path, n_acc, bonus, status = outs
        slots = slots if slots is not None else torch.empty((B, max_path), dtype=torch.int32, device=dev)
        commit_status = commit_status if commit_status is not None else torch.empty(B, dtype=torch.int32, device=dev)
        ws = workspace if workspace is not None else self.workspace(max(B, 1), T, 1, 1, 64)
        tree = _Tree(B, T, parent.data_ptr(), None)
        c = cache._c()
        st = self.lib.reader_accept_commit(self._h, ctypes.byref(tree), _ptr(node_tokens), _ptr(logits), vocab,
                                           _ptr(target_ids), int(max_path), ctypes.byref(c), _ptr(k_tree), _ptr(v_tree),
                                           int(bool(update_seq_lens)), _ptr(path), _ptr(n_acc), _ptr(bonus), _ptr(slots),
                                           _ptr(ws), ws.numel(), _ptr(status), _ptr(commit_status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_accept_commit")
        return {"path": path, "n_acc": n_acc, "bonus": bonus, "status": status, "target_ids": target_ids,
                "slots": slots, "commit_status": commit_status}

    def accept_noalloc(self, parent: torch.Tensor, node_tokens: torch.Tensor, max_path: int, logits: torch.Tensor,
                       target_ids: Optional[torch.Tensor] = None, outs=None):
        """reader_accept_noalloc: acceptance from target logits without a workspace.  For hosts that
        cannot allocate device memory when they call; the scan's scratch is a fixed 2 MiB array inside
        the library, which limits batch * n_nodes to NOALLOC_MAX_ROWS and makes concurrent calls on
        different streams race.  When ``target_ids`` and ``outs`` are given this wrapper allocates nothing either."""
        _dev(parent, torch.int32, "parent"); _dev(node_tokens, torch.int32, "node_tokens")
        _dev(logits, torch.float32, "logits")
        B, T = parent.shape
        dev = parent.device
        if target_ids is None:
            target_ids = torch.empty((B, T), dtype=torch.int32, device=dev)
        _dev(target_ids, torch.int32, "target_ids")
        if outs is None:
            outs = (torch.empty((B, max_path), dtype=torch.int32, device=dev),
                    torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev),
                    torch.empty(B, dtype=torch.int32, device=dev))
        path, n_acc, bonus, status = outs
        tree = _Tree(B, T, parent.data_ptr(), None)
        st = self.lib.reader_accept_noalloc(self._h, ctypes.byref(tree), _ptr(node_tokens), _ptr(logits),
                                            logits.shape[-1], _ptr(target_ids), int(max_path), _ptr(path),
                                            _ptr(n_acc), _ptr(bonus), _ptr(status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_accept_noalloc")
        return {"path": path, "n_acc": n_acc, "bonus": bonus, "status": status, "target_ids": target_ids}

    def sample_targets(self, parent: torch.Tensor, logits: torch.Tensor, uniforms: torch.Tensor, temperature: float,
                       target_ids: Optional[torch.Tensor] = None, top_k: int = 0, top_p: float = 1.0) -> torch.Tensor:
        """reader_sample_targets: per-node target ids of the temperature-sampling policy with one coupled
        uniform per tree level (feed the result to accept(target_ids=...))."""
        _dev(parent, torch.int32, "parent"); _dev(logits, torch.float32, "logits"); _dev(uniforms, torch.float32, "uniforms")
        B, T = parent.shape
        if target_ids is None:
            target_ids = torch.empty((B, T), dtype=torch.int32, device=parent.device)
        tree = _Tree(B, T, parent.data_ptr(), None)
        st = self.lib.reader_sample_targets(self._h, ctypes.byref(tree), _ptr(logits), logits.shape[-1], _ptr(uniforms),
                                            float(temperature), int(top_k), float(top_p), _ptr(target_ids), _stream())
        if st != OK:
            raise ReaderError(st, "reader_sample_targets")
        return target_ids

    def kv_commit_layers(self, caches, k_trees, v_trees, path: torch.Tensor, n_acc: torch.Tensor,
                         update_seq_lens: bool = True, slots: Optional[torch.Tensor] = None,
                         status: Optional[torch.Tensor] = None):
        """reader_kv_commit_layers: the accepted rows of every layer (lists of KvCache sharing page_table and
        seq_lens, and of tree K / V tensors) committed in one launch."""
        n = len(caches)
        for t in list(k_trees) + list(v_trees):
            _dev(t, torch.bfloat16, "tree K/V")
        _dev(path, torch.int32, "path"); _dev(n_acc, torch.int32, "n_acc")
        B, T = k_trees[0].shape[:2]
        max_path = path.shape[1]
        slots = slots if slots is not None else torch.empty((B, max_path), dtype=torch.int32, device=path.device)
        status = status if status is not None else torch.empty(B, dtype=torch.int32, device=path.device)
        c_arr = (_KvCache * n)(*[c._c() for c in caches])
        k_arr = (c_void_p * n)(*[t.data_ptr() for t in k_trees])
        v_arr = (c_void_p * n)(*[t.data_ptr() for t in v_trees])
        st = self.lib.reader_kv_commit_layers(self._h, c_arr, k_arr, v_arr, n, B, T, _ptr(path), _ptr(n_acc), max_path,
                                              int(bool(update_seq_lens)), _ptr(slots), _ptr(status), _stream())
        if st != OK:
            raise ReaderError(st, "reader_kv_commit_layers")
        return slots, status

    def kv_rearrange(self, k: torch.Tensor, v: torch.Tensor, valid: torch.Tensor,
                     lengths: Optional[torch.Tensor] = None) -> torch.Tensor:
        """reader_kv_rearrange: Algorithm 4 on a padded batch cache k, v [B, Hkv, cap, D] with a validity mask
        [B, cap] (uint8); compacts in place, rewrites the mask, returns the lengths."""
        _dev(k, torch.bfloat16, "k"); _dev(v, torch.bfloat16, "v"); _dev(valid, torch.uint8, "valid")
        B, Hkv, cap, D = k.shape
        if lengths is None:
            lengths = torch.empty(B, dtype=torch.int32, device=k.device)
        st = self.lib.reader_kv_rearrange(self._h, _ptr(k), _ptr(v), B, Hkv, cap, D, _ptr(valid), _ptr(lengths), _stream())
        if st != OK:
            raise ReaderError(st, "reader_kv_rearrange")
        return lengths

    def kv_commit(self, cache: KvCache, k_tree: torch.Tensor, v_tree: torch.Tensor, path: torch.Tensor,
                  n_acc: torch.Tensor, update_seq_lens: bool = True, slots: Optional[torch.Tensor] = None,
                  status: Optional[torch.Tensor] = None):
        _dev(k_tree, torch.bfloat16, "k_tree"); _dev(v_tree, torch.bfloat16, "v_tree")
        _dev(path, torch.int32, "path"); _dev(n_acc, torch.int32, "n_acc")
        B, T = k_tree.shape[:2]
        max_path = path.shape[1]
        slots = slots if slots is not None else torch.empty((B, max_path), dtype=torch.int32, device=path.device)
        status = status if status is not None else torch.empty(B, dtype=torch.int32, device=path.device)
        c = cache._c()
        st = self.lib.reader_kv_commit(self._h, ctypes.byref(c), _ptr(k_tree), _ptr(v_tree), B, T, _ptr(path),
                                       _ptr(n_acc), max_path, int(bool(update_seq_lens)), _ptr(slots), _ptr(status),
                                       _stream())
        if st != OK:
            raise ReaderError(st, "reader_kv_commit")
        return slots, status


# ---------------------------------------------------------------------------------------------
# moving a host workload onto the device (no arithmetic)
# ---------------------------------------------------------------------------------------------
def bf16_tensor(bits, device) -> torch.Tensor:
    """numpy uint16 bit patterns -> torch.bfloat16 tensor on `device` (reinterpretation, no rounding)."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def bf16_bits(t: torch.Tensor):
    """torch.bfloat16 tensor -> numpy uint16 bit patterns on the host."""
    import numpy as np
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


@dataclass
class DeviceWorkload:
    q: torch.Tensor
    k_tree: torch.Tensor
    v_tree: torch.Tensor
    cache: KvCache
    parent: torch.Tensor
    node_tokens: torch.Tensor
    logits: Optional[torch.Tensor]
    scale: float
    max_path: int


def to_device(w, device="cuda:0", with_logits: bool = True) -> DeviceWorkload:
    cache = KvCache(bf16_tensor(w.k_pool, device), bf16_tensor(w.v_pool, device),
                    torch.from_numpy(w.page_table).to(device), torch.from_numpy(w.seq_lens).to(device),
                    w.shared_prefix_len)
    logits = torch.from_numpy(w.logits).to(device) if (with_logits and w.logits is not None) else None
    return DeviceWorkload(bf16_tensor(w.q, device), bf16_tensor(w.k_tree, device), bf16_tensor(w.v_tree, device),
                          cache, torch.from_numpy(w.parent).to(device), torch.from_numpy(w.node_tokens).to(device),
                          logits, float(w.scale), int(w.max_path))


def padded_to_device(pc, device="cuda:0") -> PaddedCache:
    """A workloads.PaddedCache (numpy) as device tensors."""
    return PaddedCache(bf16_tensor(pc.k, device), bf16_tensor(pc.v, device), torch.from_numpy(pc.valid).to(device),
                       torch.tensor([pc.extent], dtype=torch.int32, device=device))
