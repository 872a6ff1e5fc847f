"""Thin ctypes binding of the C ABI in ``include/wg.h``.

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
Device buffers are ``torch`` tensors (PyTorch is used for device memory and streams); host
arrays are numpy.  There is no CPU fallback: if ``libwg.so`` has not been built, importing
this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libwg.so")

WG_OK = 0
WG_ERR_ARG = -1
WG_ERR_GRAMMAR = -2
WG_ERR_CAPACITY = -3
WG_ERR_TOKEN_REJECTED = -4
WG_ERR_CUDA = -5
WG_ERR_EMPTY_MASK = -6
WG_ERR_STATE = -7

WG_DTYPE_BF16 = 0
WG_DTYPE_FP32 = 1
WG_USE_CACHE = 0
WG_NO_CACHE = 1
WG_RESTART_ON_DONE = 2
WG_CACHE_DENSE = 0
WG_CACHE_COMPACT = 1
WG_ENTRY_ALLOWS = 0
WG_ENTRY_DENIES = 1

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2507_16768_b200.build` "
        "(nvcc, sm_100a). This package has no CPU fallback.")

_lib = C.CDLL(LIB_PATH)


class WgStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "cache_hits", "cache_misses", "masks_built", "rows_uncached", "tokens_rejected",
        "empty_masks", "bad_states", "cache_entries", "cache_bytes")]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


_vp, _i32, _i64, _u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32
_SIGNATURES = {
    "wg_load_vocab": (_i32, [_vp, _vp, _i32, _i32, C.POINTER(_vp)]),
    "wg_vocab_free": (None, [_vp]),
    "wg_compile_grammar": (_i32, [_vp, _i32, _vp, _i32, _vp, _i32, _vp, _i32, _i32, C.POINTER(_vp)]),
    "wg_grammar_free": (None, [_vp]),
    "wg_grammar_minimize": (_i32, [_vp, C.POINTER(_vp)]),
    "wg_template_compile": (_i32, [_vp, _i32, _vp, _i32, _vp, _i32, _vp, _i32, _i32, C.POINTER(_vp)]),
    "wg_template_info": (_i32, [_vp, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32)]),
    "wg_template_instantiate": (_i32, [_vp, C.POINTER(_vp), _i32, C.POINTER(_vp)]),
    "wg_template_free": (None, [_vp]),
    "wg_grammar_save": (_i32, [_vp, _vp, C.c_size_t, C.POINTER(C.c_size_t)]),
    "wg_grammar_load": (_i32, [C.c_char_p, C.c_size_t, C.POINTER(_vp)]),
    "wg_regex_to_optree": (_i32, [C.c_char_p, _i32, C.POINTER(_vp)]),
    "wg_optree_sizes": (_i32, [_vp, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32),
                               C.POINTER(_i32), C.POINTER(_i32)]),
    "wg_optree_copy": (_i32, [_vp, _vp, _vp, _vp, _vp]),
    "wg_optree_free": (None, [_vp]),
    "wg_compile_regex": (_i32, [C.c_char_p, _i32, C.POINTER(_vp)]),
    "wg_compile_regex_fragment": (_i32, [C.c_char_p, _i32, C.POINTER(_vp)]),
    "wg_regex_error": (C.c_char_p, []),
    "wg_grammar_info": (_i32, [_vp, C.POINTER(_i32), C.POINTER(_i32), C.POINTER(_i32),
                               C.POINTER(_i32), C.POINTER(C.c_uint64)]),
    "wg_grammar_step": (_i32, [_vp, _i32, _i32]),
    "wg_grammar_forced_token": (_i32, [_vp, _i32, C.POINTER(_i32), C.POINTER(_i32)]),
    "wg_ctx_create": (_i32, [_vp, _i32, _i32, C.POINTER(_vp)]),
    "wg_ctx_create_ex": (_i32, [_vp, _i32, _i32, _i32, C.c_size_t, C.POINTER(_vp)]),
    "wg_ctx_free": (None, [_vp]),
    "wg_cache_entry_read": (_i32, [_vp, _i32, _i32, C.POINTER(_i32), C.POINTER(_i32), _vp, _i32,
                                   C.POINTER(_i64), _vp]),
    "wg_ctx_add_grammar": (_i32, [_vp, _vp, C.POINTER(_i32)]),
    "wg_ctx_remove_grammar": (_i32, [_vp, _i32]),
    "wg_cache_prewarm": (_i32, [_vp, _i32, _vp]),
    "wg_cache_clear": (_i32, [_vp, _vp]),
    "wg_get_stats": (_i32, [_vp, C.POINTER(WgStats), _vp]),
    "wg_reset_stats": (_i32, [_vp, _vp]),
    "wg_mask_cache_lookup": (_i32, [_vp, _vp, _vp, _i32, _vp, _vp]),
    "wg_build_masks": (_i32, [_vp, _vp, _vp, _i32, _vp, _i64, _u32, _vp]),
    "wg_apply_mask": (_i32, [_vp, _i32, _i64, _vp, _i64, _i32, _i32, _vp, _vp, _vp]),
    "wg_apply_workspace_bytes": (C.c_size_t, [_i32]),
    "wg_apply_mask_noalloc": (_i32, [_vp, _i32, _i64, _vp, _i64, _i32, _i32, _vp, _vp]),
    "wg_advance": (_i32, [_vp, _vp, _vp, _vp, _i32, _vp, _u32, _vp]),
    "wg_decode_step": (_i32, [_vp, _vp, _vp, _i32, _vp, _i32, _i64, _vp, _i64, _vp, _vp, _u32, _vp]),
    "wg_decode_step_shard": (_i32, [_vp, _vp, _vp, _i32, _vp, _i32, _i64, _vp, _i64, _i32, _i32, _vp,
                                    _u32, _vp]),
    "wg_advance_keys": (_i32, [_vp, _vp, _vp, _vp, _i32, _vp, _vp, _u32, _vp]),
    "wg_step_graph_create": (_i32, [_vp, _vp, _vp, _i32, _vp, _i32, _i64, _vp, _i64, _vp, _vp, _u32,
                                    C.POINTER(_vp)]),
    "wg_step_graph_launch": (_i32, [_vp, _vp]),
    "wg_step_graph_free": (None, [_vp]),
    "wg_decode_step_host": (_i32, [_vp, _vp, _vp, _i32, _vp, _vp, _i32, _i64, _vp, _i64, _vp, _vp,
                                   _vp, _u32, _vp]),
    "wg_ctx_set_timing": (_i32, [_vp, _i32]),
    "wg_ctx_get_timing": (_i32, [_vp, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                 C.POINTER(_i64)]),
    "wg_ctx_count_build_work": (_i32, [_vp, _i32]),
    "wg_get_build_work": (_i32, [_vp, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64), _vp]),
    "wg_strerror": (C.c_char_p, [_i32]),
    "wg_last_cuda_error": (_i32, []),
    "wg_kernel_launch_count": (_i64, []),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _f = getattr(_lib, _name)
    _f.restype = _res
    _f.argtypes = _args

EXPORTED = tuple(_SIGNATURES)


class WgError(RuntimeError):
    def __init__(self, status: int, where: str):
        msg = _lib.wg_strerror(int(status)).decode()
        if status == WG_ERR_CUDA:
            msg += f" (cudaError {_lib.wg_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")
        self.status = int(status)


def _check(status: int, where: str) -> None:
    if status != WG_OK:
        raise WgError(status, where)


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _device_of(ctx):
    """Index of the device a context (or None: any device) lives on."""
    return None if ctx is None else getattr(ctx, "device", None)


def _dev_ptr(t, dtype=None, what: str = "tensor", device=None):
    """Raw device pointer of a torch CUDA tensor (None passes through)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"{what} must be a CUDA tensor")
    if dtype is not None and t.dtype not in (dtype if isinstance(dtype, tuple) else (dtype,)):
        raise TypeError(f"{what} has dtype {t.dtype}")
    if device is not None and t.device.index != device:
        raise ValueError(f"{what} lives on cuda:{t.device.index}, the context on cuda:{device}")
    return C.c_void_p(t.data_ptr())


def _vec(t, n: int, dtype, what: str, device=None):
    """Pointer of a contiguous 1-D device array that holds at least ``n`` elements: the kernels
    index these arrays by row number without any further check."""
    if t is None:
        return None
    p = _dev_ptr(t, dtype, what, device)
    if t.dim() != 1 or not t.is_contiguous():
        raise ValueError(f"{what} must be a contiguous 1-D tensor")
    if t.numel() < n:
        raise ValueError(f"{what} holds {t.numel()} elements, the batch has {n} rows")
    return p


def _mat(t, rows: int, cols: int, dtype, what: str, device=None):
    """(pointer, row stride) of a 2-D device array with unit inner stride that holds at least
    ``rows`` rows of ``cols`` elements."""
    p = _dev_ptr(t, dtype, what, device)
    _, stride = _rows(t, what)
    if t.shape[0] < rows or t.shape[1] < cols:
        raise ValueError(f"{what} is {tuple(t.shape)}, at least ({rows}, {cols}) is needed")
    return p, stride


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def kernel_launch_count() -> int:
    return int(_lib.wg_kernel_launch_count())


class Vocab:
    """wg_load_vocab: copies a CSR vocabulary (numpy, host) to the current device."""

    def __init__(self, offsets: np.ndarray, data: np.ndarray, eos_id: int):
        self._offsets = np.ascontiguousarray(offsets, np.uint32)
        self._data = np.ascontiguousarray(data, np.uint8)
        self.V = int(self._offsets.shape[0] - 1)
        self.W = (self.V + 31) // 32
        self.eos_id = int(eos_id)
        h = _vp()
        _check(_lib.wg_load_vocab(_np_ptr(self._offsets), _np_ptr(self._data), self.V, self.eos_id,
                                  C.byref(h)), "wg_load_vocab")
        self.handle = h
        import torch
        self.device = torch.cuda.current_device()     # wg_load_vocab uploads to the current device

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.wg_vocab_free(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


class RegexTree:
    """The operator tree of a regular expression as flat arrays (wg_regex_to_optree)."""

    def __init__(self, pattern):
        if isinstance(pattern, str):
            pattern = pattern.encode("utf-8")
        h = _vp()
        rc = _lib.wg_regex_to_optree(pattern, len(pattern), C.byref(h))
        if rc != WG_OK:
            raise WgError(rc, "wg_regex_to_optree: " + _lib.wg_regex_error().decode())
        try:
            n = [_i32() for _ in range(5)]
            _check(_lib.wg_optree_sizes(h, *[C.byref(x) for x in n]), "wg_optree_sizes")
            self.nodes = np.zeros((n[0].value, 8), np.int32)
            self.children = np.zeros(n[1].value, np.int32)
            self.sets = np.zeros((n[2].value, 9), np.uint32)
            self.data = np.zeros(n[3].value, np.uint8)
            self.root = n[4].value
            _check(_lib.wg_optree_copy(h, _np_ptr(self.nodes), _np_ptr(self.children),
                                       _np_ptr(self.sets), _np_ptr(self.data)), "wg_optree_copy")
        finally:
            _lib.wg_optree_free(h)

    @property
    def n_nodes(self) -> int:
        return int(self.nodes.shape[0])


class Grammar:
    """wg_compile_grammar: lowers a flat operator tree to a byte-level table (host side).

    ``Grammar.from_regex(pattern)`` goes through wg_compile_regex instead.
    """

    def __init__(self, flat=None, _handle=None):
        if _handle is None:
            nodes = np.ascontiguousarray(flat.nodes, np.int32)
            children = np.ascontiguousarray(flat.children, np.int32)
            sets = np.ascontiguousarray(flat.sets, np.uint32)
            data = np.ascontiguousarray(flat.data, np.uint8)
            _handle = _vp()
            _check(_lib.wg_compile_grammar(_np_ptr(nodes), nodes.shape[0], _np_ptr(children),
                                           children.shape[0], _np_ptr(sets), sets.shape[0],
                                           _np_ptr(data), data.shape[0], int(flat.root),
                                           C.byref(_handle)), "wg_compile_grammar")
        h = _handle
        self.handle = h
        n, s, d, c, hs = _i32(), _i32(), _i32(), _i32(), C.c_uint64()
        _check(_lib.wg_grammar_info(h, C.byref(n), C.byref(s), C.byref(d), C.byref(c), C.byref(hs)),
               "wg_grammar_info")
        self.n_states, self.start_state, self.done_state = n.value, s.value, d.value
        self.n_classes, self.content_hash = c.value, hs.value

    @classmethod
    def from_regex(cls, pattern, fragment: bool = False) -> "Grammar":
        """wg_compile_regex, or wg_compile_regex_fragment for a template argument."""
        if isinstance(pattern, str):
            pattern = pattern.encode("utf-8")
        h = _vp()
        fn = _lib.wg_compile_regex_fragment if fragment else _lib.wg_compile_regex
        rc = fn(pattern, len(pattern), C.byref(h))
        if rc != WG_OK:
            raise WgError(rc, "wg_compile_regex: " + _lib.wg_regex_error().decode())
        return cls(_handle=h)

    def save(self) -> bytes:
        """wg_grammar_save: the compiled table as a blob for wg_grammar_load."""
        need = C.c_size_t()
        _lib.wg_grammar_save(self.handle, None, 0, C.byref(need))
        buf = C.create_string_buffer(need.value)
        _check(_lib.wg_grammar_save(self.handle, buf, need.value, C.byref(need)), "wg_grammar_save")
        return buf.raw

    @classmethod
    def load(cls, blob: bytes) -> "Grammar":
        h = _vp()
        _check(_lib.wg_grammar_load(blob, len(blob), C.byref(h)), "wg_grammar_load")
        return cls(_handle=h)

    def minimized(self) -> "Grammar":
        """wg_grammar_minimize: the same language with equivalent states merged."""
        h = _vp()
        _check(_lib.wg_grammar_minimize(self.handle, C.byref(h)), "wg_grammar_minimize")
        return Grammar(_handle=h)

    def step(self, state: int, symbol: int) -> int:
        return int(_lib.wg_grammar_step(self.handle, int(state), int(symbol)))

    def forced_token(self, state: int):
        """(token id, next state) if ``state`` belongs to a token-level Write, else None."""
        tok, nxt = _i32(), _i32()
        if _lib.wg_grammar_forced_token(self.handle, int(state), C.byref(tok), C.byref(nxt)):
            return tok.value, nxt.value
        return None

    def step_token(self, state: int, token: int, symbols) -> int:
        """Host-side state after a whole token (``symbols`` = its bytes, or [256] for EOS)."""
        forced = self.forced_token(state)
        if forced is not None:
            return forced[1] if token == forced[0] else 0
        return self.walk(state, symbols)

    def walk(self, state: int, symbols) -> int:
        for s in symbols:
            state = self.step(state, s)
        return state

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.wg_grammar_free(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


class Template:
    """wg_template_compile: an operator tree with holes, lowered once; ``instantiate`` splices
    one compiled grammar per argument into the holes (wg_template_instantiate)."""

    def __init__(self, flat):
        nodes = np.ascontiguousarray(flat.nodes, np.int32)
        children = np.ascontiguousarray(flat.children, np.int32)
        sets = np.ascontiguousarray(flat.sets, np.uint32)
        data = np.ascontiguousarray(flat.data, np.uint8)
        h = _vp()
        _check(_lib.wg_template_compile(_np_ptr(nodes), nodes.shape[0], _np_ptr(children),
                                        children.shape[0], _np_ptr(sets), sets.shape[0],
                                        _np_ptr(data), data.shape[0], int(flat.root), C.byref(h)),
               "wg_template_compile")
        self.handle = h
        n, k, a = _i32(), _i32(), _i32()
        _check(_lib.wg_template_info(h, C.byref(n), C.byref(k), C.byref(a)), "wg_template_info")
        self.n_states, self.n_holes, self.n_args = n.value, k.value, a.value

    def instantiate(self, args) -> Grammar:
        args = list(args)
        arr = (_vp * max(1, len(args)))(*[g.handle for g in args])
        h = _vp()
        _check(_lib.wg_template_instantiate(self.handle, arr, len(args), C.byref(h)),
               "wg_template_instantiate")
        return Grammar(_handle=h)

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.wg_template_free(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


class Context:
    """wg_ctx: device tables, the mask cache and per-batch scratch."""

    def __init__(self, vocab: Vocab, cache_capacity: int, max_batch: int,
                 cache_mode: int = WG_CACHE_DENSE, arena_bytes: int = 0):
        self.vocab = vocab
        self.max_batch = int(max_batch)
        self.device = vocab.device
        h = _vp()
        if cache_mode == WG_CACHE_DENSE and not arena_bytes:
            _check(_lib.wg_ctx_create(vocab.handle, int(cache_capacity), int(max_batch),
                                      C.byref(h)), "wg_ctx_create")
        else:
            _check(_lib.wg_ctx_create_ex(vocab.handle, int(cache_capacity), int(max_batch),
                                         int(cache_mode), int(arena_bytes), C.byref(h)),
                   "wg_ctx_create_ex")
        self.handle = h

    def cache_entry(self, grammar_id: int, state: int, stream=None):
        """wg_cache_entry_read: (kind, sorted token ids, device bytes) of one compact cache
        entry, or None when the state is not cached."""
        kind, n, nbytes = _i32(), _i32(), _i64()
        ids = np.zeros(self.vocab.V, np.int32)
        _check(_lib.wg_cache_entry_read(self.handle, int(grammar_id), int(state), C.byref(kind),
                                        C.byref(n), _np_ptr(ids), ids.shape[0], C.byref(nbytes),
                                        _stream_ptr(stream)), "wg_cache_entry_read")
        if kind.value < 0:
            return None
        return kind.value, ids[:n.value].copy(), int(nbytes.value)

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.wg_ctx_free(self.handle)
            self.handle = None

    def __del__(self):
        self.close()

    def add_grammar(self, grammar: Grammar) -> int:
        gid = _i32()
        _check(_lib.wg_ctx_add_grammar(self.handle, grammar.handle, C.byref(gid)),
               "wg_ctx_add_grammar")
        return gid.value

    def remove_grammar(self, grammar_id: int) -> None:
        """Frees the grammar's tables and cached masks; the id goes to a grammar added later."""
        _check(_lib.wg_ctx_remove_grammar(self.handle, int(grammar_id)), "wg_ctx_remove_grammar")

    def cache_prewarm(self, grammar_id: int, stream=None) -> None:
        _check(_lib.wg_cache_prewarm(self.handle, int(grammar_id), _stream_ptr(stream)),
               "wg_cache_prewarm")

    def cache_clear(self, stream=None) -> None:
        _check(_lib.wg_cache_clear(self.handle, _stream_ptr(stream)), "wg_cache_clear")

    def stats(self, stream=None) -> dict:
        st = WgStats()
        _check(_lib.wg_get_stats(self.handle, C.byref(st), _stream_ptr(stream)), "wg_get_stats")
        return st.as_dict()

    def set_timing(self, enable: bool) -> None:
        _check(_lib.wg_ctx_set_timing(self.handle, int(bool(enable))), "wg_ctx_set_timing")

    def get_timing(self) -> dict:
        """Summed kernel milliseconds of the steps recorded since the last read."""
        b, a, n = C.c_double(), C.c_double(), _i64()
        _check(_lib.wg_ctx_get_timing(self.handle, C.byref(b), C.byref(a), C.byref(n)),
               "wg_ctx_get_timing")
        return {"build_ms": b.value, "apply_ms": a.value, "steps": int(n.value)}

    def count_build_work(self, enable: bool) -> None:
        _check(_lib.wg_ctx_count_build_work(self.handle, int(bool(enable))),
               "wg_ctx_count_build_work")

    def build_work(self, stream=None) -> dict:
        """Work counted by the build kernel's counting variant since the last reset_stats."""
        q, l, m = _i64(), _i64(), _i64()
        _check(_lib.wg_get_build_work(self.handle, C.byref(q), C.byref(l), C.byref(m),
                                      _stream_ptr(stream)), "wg_get_build_work")
        return {"tokens_walked": q.value, "table_lookups": l.value, "mask_words_read": m.value}

    def reset_stats(self, stream=None) -> None:
        _check(_lib.wg_reset_stats(self.handle, _stream_ptr(stream)), "wg_reset_stats")


def _logits_dtype(logits) -> int:
    import torch
    if logits.dtype == torch.bfloat16:
        return WG_DTYPE_BF16
    if logits.dtype == torch.float32:
        return WG_DTYPE_FP32
    raise TypeError(f"logits must be bfloat16 or float32, not {logits.dtype}")


def _rows(t, what: str):
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError(f"{what} must be 2-D with unit inner stride")
    return t.shape[0], t.stride(0)


def wg_mask_cache_lookup(ctx: Context, gid, sid, slot, stream=None) -> None:
    import torch
    B, dev = gid.shape[0], _device_of(ctx)
    _check(_lib.wg_mask_cache_lookup(ctx.handle, _vec(gid, B, torch.int32, "gid", dev),
                                     _vec(sid, B, torch.int32, "sid", dev), B,
                                     _vec(slot, B, torch.int32, "slot", dev), _stream_ptr(stream)),
           "wg_mask_cache_lookup")


def wg_build_masks(ctx: Context, gid, sid, bitmask, flags: int = WG_USE_CACHE, stream=None) -> None:
    import torch
    B, dev = bitmask.shape[0], _device_of(ctx)
    mask, stride = _mat(bitmask, B, ctx.vocab.W, (torch.int32, torch.uint32), "bitmask", dev)
    _check(_lib.wg_build_masks(ctx.handle, _vec(gid, B, torch.int32, "gid", dev),
                               _vec(sid, B, torch.int32, "sid", dev), B, mask, stride,
                               int(flags), _stream_ptr(stream)), "wg_build_masks")


def _apply_args(logits, bitmask, V: int, argmax_out):
    """Checked (logits pointer, dtype, stride, mask pointer, mask stride, B, token pointer)."""
    import torch
    if logits.dim() != 2:
        raise ValueError("logits must be 2-D with unit inner stride")
    B, V = logits.shape[0], int(V)
    dev = logits.device.index if logits.is_cuda else None
    lp, stride = _mat(logits, B, V, None, "logits", dev)
    mp, mstride = _mat(bitmask, B, (V + 31) // 32, (torch.int32, torch.uint32), "bitmask", dev)
    return lp, _logits_dtype(logits), stride, mp, mstride, B, V, \
        _vec(argmax_out, B, torch.int32, "argmax_out", dev), dev


def wg_apply_mask(logits, bitmask, V: int, argmax_out=None, workspace=None, stream=None) -> None:
    lp, dtype, stride, mp, mstride, B, V, tok, dev = _apply_args(logits, bitmask, V, argmax_out)
    ws = _dev_ptr(workspace, None, "workspace", dev)
    if argmax_out is not None:
        need = wg_apply_workspace_bytes(B)
        if workspace is None or not workspace.is_contiguous() or \
                workspace.numel() * workspace.element_size() < need:
            raise ValueError(f"workspace must be a contiguous device buffer of {need} bytes")
    _check(_lib.wg_apply_mask(lp, dtype, stride, mp, mstride, B, V, tok, ws, _stream_ptr(stream)),
           "wg_apply_mask")


WG_NOALLOC_MAX_ROWS = 4096


def wg_apply_mask_noalloc(logits, bitmask, V: int, argmax_out, stream=None) -> None:
    """Mask + greedy argmax for callers that may not allocate device memory.

    Same results as ``wg_apply_mask`` with ``argmax_out``; the scratch is a fixed 32 KB array
    inside the library, so at most ``WG_NOALLOC_MAX_ROWS`` rows per call, and calls that can
    overlap on the GPU must not be issued (they share that array).
    """
    if argmax_out is None:
        raise ValueError("argmax_out is required")
    lp, dtype, stride, mp, mstride, B, V, tok, _ = _apply_args(logits, bitmask, V, argmax_out)
    _check(_lib.wg_apply_mask_noalloc(lp, dtype, stride, mp, mstride, B, V, tok,
                                      _stream_ptr(stream)), "wg_apply_mask_noalloc")


def wg_apply_workspace_bytes(B: int) -> int:
    return int(_lib.wg_apply_workspace_bytes(int(B)))


def wg_advance(ctx: Context, gid, sid, token, status=None, flags: int = 0, stream=None) -> None:
    import torch
    B, dev = gid.shape[0], _device_of(ctx)
    _check(_lib.wg_advance(ctx.handle, _vec(gid, B, torch.int32, "gid", dev),
                           _vec(sid, B, torch.int32, "sid", dev),
                           _vec(token, B, torch.int32, "token", dev), B,
                           _vec(status, B, torch.int32, "status", dev), int(flags),
                           _stream_ptr(stream)), "wg_advance")


def _step_args(ctx: Context, gid, sid, logits, n_cols: int, bitmask, token_out, status):
    """The checked arrays of one decode step over ``logits.shape[0]`` rows."""
    import torch
    if logits.dim() != 2:
        raise ValueError("logits must be 2-D with unit inner stride")
    B, dev = logits.shape[0], _device_of(ctx)
    lp, stride = _mat(logits, B, n_cols, None, "logits", dev)
    mp, mstride = _mat(bitmask, B, ctx.vocab.W, (torch.int32, torch.uint32), "bitmask", dev)
    return (_vec(gid, B, torch.int32, "gid", dev), _vec(sid, B, torch.int32, "sid", dev), B, lp,
            _logits_dtype(logits), stride, mp, mstride,
            _vec(token_out, B, torch.int32, "token_out", dev),
            _vec(status, B, torch.int32, "status", dev))


def wg_decode_step(ctx: Context, gid, sid, logits, bitmask, token_out, status=None,
                   flags: int = WG_USE_CACHE, stream=None) -> None:
    """One decode step.  With ``token_out`` None the step only masks (no argmax, no advance): the
    caller samples from the masked logits and calls ``wg_advance``."""
    g, s, B, lp, dtype, stride, mp, mstride, tok, st = _step_args(
        ctx, gid, sid, logits, ctx.vocab.V, bitmask, token_out, status)
    if tok is None and (st is not None or int(flags) & WG_RESTART_ON_DONE):
        raise ValueError("a step without token_out advances nothing: no status, no WG_RESTART_ON_DONE")
    _check(_lib.wg_decode_step(ctx.handle, g, s, B, lp, dtype, stride, mp, mstride, tok, st,
                               int(flags), _stream_ptr(stream)), "wg_decode_step")


WG_SHARD_ALIGN = 8192


def wg_decode_step_shard(ctx: Context, gid, sid, logits_shard, bitmask, v_begin: int, v_end: int,
                         best_keys, flags: int = WG_USE_CACHE, stream=None) -> None:
    """The decode step on the vocabulary slice [v_begin, v_end); ``best_keys`` (int64, B) gets
    the packed per-row maxima to be MAX-reduced over the GPUs that hold the other slices."""
    import torch
    g, s, B, lp, dtype, stride, mp, mstride, _, _ = _step_args(
        ctx, gid, sid, logits_shard, max(int(v_end) - int(v_begin), 0), bitmask, None, None)
    _check(_lib.wg_decode_step_shard(
        ctx.handle, g, s, B, lp, dtype, stride, mp, mstride, int(v_begin), int(v_end),
        _vec(best_keys, B, torch.int64, "best_keys", _device_of(ctx)), int(flags),
        _stream_ptr(stream)), "wg_decode_step_shard")


def wg_advance_keys(ctx: Context, gid, sid, best_keys, token_out, status=None, flags: int = 0,
                    stream=None) -> None:
    import torch
    B, dev = gid.shape[0], _device_of(ctx)
    _check(_lib.wg_advance_keys(ctx.handle, _vec(gid, B, torch.int32, "gid", dev),
                                _vec(sid, B, torch.int32, "sid", dev),
                                _vec(best_keys, B, torch.int64, "best_keys", dev), B,
                                _vec(token_out, B, torch.int32, "token_out", dev),
                                _vec(status, B, torch.int32, "status", dev), int(flags),
                                _stream_ptr(stream)), "wg_advance_keys")


class StepPlan:
    """A wg_decode_step call with everything but the logits marshalled once.

    The per-call work of the binding (pointer extraction, dtype and shape checks) costs more
    than a small decode step takes on the GPU; a plan does it once for buffers that stay put
    (ids, states, bitmask, tokens, status) and only takes the logits tensor per call.
    """

    def __init__(self, ctx: Context, gid, sid, bitmask, token_out, status=None,
                 flags: int = WG_USE_CACHE, stream=None):
        import torch
        self._keep = (ctx, gid, sid, bitmask, token_out, status)
        self.B, dev = bitmask.shape[0], _device_of(ctx)
        if gid.shape[0] != self.B or sid.shape[0] != self.B or token_out.shape[0] != self.B:
            raise ValueError("gid, sid, token_out and bitmask disagree on the batch size")
        self._ctx = ctx.handle
        self._V, self._device = ctx.vocab.V, dev
        self._gid = _vec(gid, self.B, torch.int32, "gid", dev)
        self._sid = _vec(sid, self.B, torch.int32, "sid", dev)
        self._mask, self._mstride = _mat(bitmask, self.B, ctx.vocab.W, (torch.int32, torch.uint32),
                                         "bitmask", dev)
        self._tok = _vec(token_out, self.B, torch.int32, "token_out", dev)
        self._status = _vec(status, self.B, torch.int32, "status", dev)
        self._flags = int(flags)
        self._stream = _stream_ptr(stream)
        self._dtypes = {torch.bfloat16: WG_DTYPE_BF16, torch.float32: WG_DTYPE_FP32}
        self._fn = _lib.wg_decode_step

    def __call__(self, logits) -> None:
        if logits.dim() != 2 or logits.shape[0] != self.B or logits.shape[1] < self._V \
                or logits.stride(1) != 1 or not logits.is_cuda \
                or (self._device is not None and logits.device.index != self._device):
            raise ValueError("logits must be a tensor [B, V] with unit inner stride on the "
                             "context's device")
        rc = self._fn(self._ctx, self._gid, self._sid, self.B, logits.data_ptr(),
                      self._dtypes[logits.dtype], logits.stride(0), self._mask, self._mstride,
                      self._tok, self._status, self._flags, self._stream)
        if rc != WG_OK:
            raise WgError(rc, "wg_decode_step")


class StepGraph:
    """wg_step_graph: one decode step recorded as a CUDA graph for fixed buffers."""

    def __init__(self, ctx: Context, gid, sid, logits, bitmask, token_out, status=None,
                 flags: int = WG_USE_CACHE):
        self._keep = (ctx, gid, sid, logits, bitmask, token_out, status)
        g, s, B, lp, dtype, stride, mp, mstride, tok, st = _step_args(
            ctx, gid, sid, logits, ctx.vocab.V, bitmask, token_out, status)
        if tok is None:
            raise ValueError("token_out is required")
        h = _vp()
        _check(_lib.wg_step_graph_create(ctx.handle, g, s, B, lp, dtype, stride, mp, mstride, tok, st,
                                         int(flags), C.byref(h)), "wg_step_graph_create")
        self.handle = h
        self._launch = _lib.wg_step_graph_launch

    def launch(self, stream=None) -> None:
        rc = self._launch(self.handle, _stream_ptr(stream))
        if rc != WG_OK:
            raise WgError(rc, "wg_step_graph_launch")

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.wg_step_graph_free(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


def wg_decode_step_host(ctx: Context, gid, sid, logits_host, logits_dev, bitmask, token_dev,
                        token_host, status=None, flags: int = WG_USE_CACHE, stream=None) -> None:
    """logits_host / token_host are CPU tensors (pinned for asynchronous copies)."""
    g, s, B, lp, dtype, stride, mp, mstride, tok, st = _step_args(
        ctx, gid, sid, logits_dev, ctx.vocab.V, bitmask, token_dev, status)
    if tok is None:
        raise ValueError("token_dev is required")
    if logits_host.is_cuda or token_host.is_cuda or not logits_host.is_contiguous() \
            or not token_host.is_contiguous():
        raise TypeError("logits_host and token_host must be contiguous CPU tensors")
    if logits_host.dim() != 2 or logits_host.shape[0] < B or logits_host.shape[1] != ctx.vocab.V \
            or logits_host.dtype != logits_dev.dtype:
        raise ValueError("logits_host must hold B rows of V elements of the device dtype")
    if token_host.numel() < B or token_host.element_size() != 4:
        raise ValueError("token_host must hold B 32-bit integers")
    _check(_lib.wg_decode_step_host(
        ctx.handle, g, s, B, C.c_void_p(logits_host.data_ptr()), lp, dtype, stride, mp, mstride,
        tok, C.c_void_p(token_host.data_ptr()), st, int(flags), _stream_ptr(stream)),
        "wg_decode_step_host")
