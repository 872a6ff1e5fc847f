"""ctypes front end of the CPU checker (``wg_oracle.c``).

TEST INFRASTRUCTURE.  Only the tests, the smoke entry and the CPU-baseline leg of the
benchmark may import this package; the product (``paper_2507_16768_b200``) never does, and
this package never imports the product.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wg_oracle.c")
_LIB = os.path.join(_HERE, "libwg_oracle.so")

DONE = (-1, 0)
DEAD_NODE = -2
ERR_ARG = -1
ERR_GRAMMAR = -2
ERR_REJECTED = -4
EOS_SYMBOL = 256


def build(force: bool = False) -> str:
    """Compile the checker with gcc (OpenMP only spreads independent rows over threads)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-Wall", "-Wextra", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.wgo_tree_create.argtypes = [vp, i32, vp, i32, vp, i32, vp, i32, i32, C.POINTER(vp)]
        L.wgo_tree_create.restype = C.c_int
        L.wgo_tree_free.argtypes = [vp]
        L.wgo_tree_free.restype = None
        L.wgo_start.argtypes = [vp, vp]
        L.wgo_start.restype = None
        L.wgo_step.argtypes = [vp, vp, i32, vp]
        L.wgo_step.restype = None
        L.wgo_mask.argtypes = [vp, vp, vp, i32, i32, vp, vp]
        L.wgo_mask.restype = None
        L.wgo_masks.argtypes = [vp, vp, vp, i32, i32, vp, i32, vp, i64, i32]
        L.wgo_masks.restype = None
        for name in ("wgo_apply_f32", "wgo_apply_bf16"):
            f = getattr(L, name)
            f.argtypes = [vp, i64, vp, i64, i32, i32, i32]
            f.restype = None
        for name in ("wgo_argmax_f32", "wgo_argmax_bf16"):
            f = getattr(L, name)
            f.argtypes = [vp, i64, vp, i64, i32, i32, vp]
            f.restype = None
        L.wgo_advance.argtypes = [vp, vp, vp, i32, i32, vp, i32]
        L.wgo_advance.restype = C.c_int
        L.wgo_max_threads.argtypes = []
        L.wgo_max_threads.restype = C.c_int
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


class OracleError(Exception):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}")
        self.code = code


class Tree:
    """An operator tree held by the checker.  Built from the flat arrays of ``flatten``."""

    def __init__(self, flat):
        self._keep = [np.ascontiguousarray(flat.nodes, np.int32),
                      np.ascontiguousarray(flat.children, np.int32),
                      np.ascontiguousarray(flat.sets, np.uint32),
                      np.ascontiguousarray(flat.data, np.uint8)]
        n, c, s, d = self._keep
        h = C.c_void_p()
        rc = lib().wgo_tree_create(_ptr(n), n.shape[0], _ptr(c), c.shape[0], _ptr(s), s.shape[0],
                                   _ptr(d), d.shape[0], int(flat.root), C.byref(h))
        if rc != 0:
            raise OracleError(rc)
        self.handle = h

    def __del__(self):
        h = getattr(self, "handle", None)
        if h and _lib is not None:
            _lib.wgo_tree_free(h)
            self.handle = None

    def start(self) -> Tuple[int, int]:
        out = np.zeros(2, np.int32)
        lib().wgo_start(self.handle, _ptr(out))
        return int(out[0]), int(out[1])

    def step(self, cursor: Tuple[int, int], symbol: int) -> Tuple[int, int]:
        cin = np.array(cursor, np.int32)
        out = np.zeros(2, np.int32)
        lib().wgo_step(self.handle, _ptr(cin), int(symbol), _ptr(out))
        return int(out[0]), int(out[1])

    def walk(self, cursor: Tuple[int, int], symbols) -> Tuple[int, int]:
        for s in symbols:
            cursor = self.step(cursor, s)
        return cursor

    def accepts(self, symbols) -> bool:
        """True iff the program has completed exactly when the symbols end."""
        return self.walk(self.start(), symbols) == DONE


def is_dead(cursor) -> bool:
    return cursor[0] == DEAD_NODE


def mask(tree: Tree, vocab, cursor) -> np.ndarray:
    W = (vocab.size + 31) // 32
    out = np.zeros(W, np.uint32)
    cin = np.array(cursor, np.int32)
    lib().wgo_mask(tree.handle, _ptr(vocab.offsets), _ptr(vocab.data), vocab.size, vocab.eos_id,
                   _ptr(cin), _ptr(out))
    return out


def masks(trees: Sequence[Tree], vocab, cursors, n_threads: int = 1,
          out: Optional[np.ndarray] = None) -> np.ndarray:
    B = len(trees)
    W = (vocab.size + 31) // 32
    if out is None:
        out = np.zeros((B, W), np.uint32)
    handles = (C.c_void_p * B)(*[t.handle for t in trees])
    cin = np.ascontiguousarray(np.asarray(cursors, np.int32).reshape(B, 2))
    lib().wgo_masks(handles, _ptr(vocab.offsets), _ptr(vocab.data), vocab.size, vocab.eos_id,
                    _ptr(cin), B, _ptr(out), out.strides[0] // 4, int(n_threads))
    return out


def apply_mask(logits: np.ndarray, bitmask: np.ndarray, V: int, n_threads: int = 1) -> None:
    """In place on raw bit patterns: uint32 (fp32) or uint16 (bf16), shape [B, >=V]."""
    assert logits.ndim == 2 and bitmask.ndim == 2 and logits.shape[0] == bitmask.shape[0]
    B = logits.shape[0]
    if logits.dtype == np.float32:
        logits = logits.view(np.uint32)
    if logits.dtype == np.uint32:
        lib().wgo_apply_f32(_ptr(logits), logits.strides[0] // 4, _ptr(bitmask),
                            bitmask.strides[0] // 4, B, V, n_threads)
    elif logits.dtype == np.uint16:
        lib().wgo_apply_bf16(_ptr(logits), logits.strides[0] // 2, _ptr(bitmask),
                             bitmask.strides[0] // 4, B, V, n_threads)
    else:
        raise TypeError(logits.dtype)


def argmax(logits: np.ndarray, bitmask: np.ndarray, V: int) -> np.ndarray:
    B = logits.shape[0]
    out = np.zeros(B, np.int32)
    if logits.dtype == np.float32:
        logits = logits.view(np.uint32)
    if logits.dtype == np.uint32:
        lib().wgo_argmax_f32(_ptr(logits), logits.strides[0] // 4, _ptr(bitmask),
                             bitmask.strides[0] // 4, B, V, _ptr(out))
    elif logits.dtype == np.uint16:
        lib().wgo_argmax_bf16(_ptr(logits), logits.strides[0] // 2, _ptr(bitmask),
                              bitmask.strides[0] // 4, B, V, _ptr(out))
    else:
        raise TypeError(logits.dtype)
    return out


def advance(tree: Tree, vocab, cursor, token: int):
    """(status, cursor'): status 0 and the new cursor, or ERR_REJECTED and the old one."""
    c = np.array(cursor, np.int32)
    rc = lib().wgo_advance(tree.handle, _ptr(vocab.offsets), _ptr(vocab.data), vocab.size,
                           vocab.eos_id, _ptr(c), int(token))
    return rc, (int(c[0]), int(c[1]))


def max_threads() -> int:
    return int(lib().wgo_max_threads())


# ---- adaptive token-set storage of a mask (paper Section 3.3) ---------------------------------
# A Wait keeps either the few tokens it refuses ("denies", when most of the vocabulary is
# accepted) or the few it accepts ("allows", when most is refused).  Written out plainly: count
# the allowed tokens among ids 0..V-1 and keep the smaller side as a sorted id list.  A tie keeps
# the allowed side.
ALLOWS = 0
DENIES = 1


def adaptive_token_set(mask_words: np.ndarray, V: int) -> Tuple[int, np.ndarray]:
    """(kind, sorted token ids) for one packed mask row."""
    allowed = [t for t in range(V) if (int(mask_words[t >> 5]) >> (t & 31)) & 1]
    if 2 * len(allowed) <= V:
        return ALLOWS, np.asarray(allowed, np.int32)
    taken = set(allowed)
    return DENIES, np.asarray([t for t in range(V) if t not in taken], np.int32)


def apply_token_set(logits: np.ndarray, kind: int, ids: np.ndarray, V: int) -> None:
    """Masks one row of raw logit bit patterns (uint16 = bf16, uint32 = fp32) in place from a
    token set: with ALLOWS every id that is not listed becomes -inf, with DENIES every listed one."""
    ninf = {np.dtype(np.uint16): 0xFF80, np.dtype(np.uint32): 0xFF800000}[logits.dtype]
    listed = set(int(t) for t in ids)
    for t in range(V):
        if (t in listed) == (kind == DENIES):
            logits[t] = ninf
