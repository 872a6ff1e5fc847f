"""Operator trees and their flat interchange format.

The operators are the compositional set of the paper's Section 3.2 (Sequence,
Wait, Write, IfElse, DoWhile) over a 257-symbol alphabet: the 256 byte values
and one end-of-sequence symbol.  This module only *describes* trees and
serialises them; it holds no matching, masking or table arithmetic.  Both the
checker under ``oracle/`` and the CUDA library consume the flat arrays
produced by :func:`flatten`, each with a parser of its own.

Flat format
-----------
``nodes``     int32 [n_nodes, 8]  rows of (kind, n_child, child_off, n_set,
                                  set_off, data_off, data_len, 0)
``children``  int32 [n_children]  node indices, -1 for an absent body
``sets``      uint32 [n_sets, 9]  257-bit symbol sets, bit ``s & 31`` of word
                                  ``s >> 5``; symbol 256 is end-of-sequence
``data``      uint8 [n_data]      literal bytes of the Write nodes
``root``      int                 index of the root node

Per kind:
  SEQUENCE  children = the parts in order
  WRITE     data     = the literal
  WAIT      sets     = [allow, deny, wait];             children = [body]
  SWITCH    sets     = [allow, deny, case_0..case_k-1]; children = [body_0..body_k-1]
  DOWHILE   sets     = [allow, deny, true, false];      children = [body]
  WAIT_UNTIL sets    = [allow, deny]; data = the string waited for; children = [body]
  WRITE_TOKENS data  = the forced token ids, 4 little-endian bytes each
  HOLE      last column of the node row = index of the argument that fills it
            (templates only: paper Section 3.1, structures that are parameterised but not
            yet instantiated)

IfElse is the two-case SWITCH: case_0 = true_waits -> if_body, case_1 =
false_waits -> else_body.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Iterable, List, Optional, Sequence as Seq, Union

import numpy as np

EOS = 256
N_SYMBOLS = 257
SET_WORDS = 9

KIND_SEQUENCE = 0
KIND_WRITE = 1
KIND_WAIT = 2
KIND_SWITCH = 3
KIND_DOWHILE = 4
KIND_WAIT_UNTIL = 5
KIND_WRITE_TOKENS = 6
KIND_HOLE = 7

SymbolsLike = Union[bytes, str, Iterable[int], "SymSet"]


class SymSet:
    """A subset of the 257-symbol alphabet."""

    __slots__ = ("bits",)

    def __init__(self, symbols: SymbolsLike = ()):  # noqa: D401
        if isinstance(symbols, SymSet):
            self.bits = symbols.bits
            return
        if isinstance(symbols, str):
            symbols = symbols.encode("utf-8")
        bits = 0
        for s in symbols:
            s = int(s)
            if not 0 <= s < N_SYMBOLS:
                raise ValueError(f"symbol {s} outside 0..256")
            bits |= 1 << s
        self.bits = bits

    @staticmethod
    def all_bytes() -> "SymSet":
        out = SymSet()
        out.bits = (1 << 256) - 1
        return out

    @staticmethod
    def range(lo: int, hi: int) -> "SymSet":
        return SymSet(range(lo, hi + 1))

    def __or__(self, other: SymbolsLike) -> "SymSet":
        out = SymSet()
        out.bits = self.bits | SymSet(other).bits
        return out

    def __sub__(self, other: SymbolsLike) -> "SymSet":
        out = SymSet()
        out.bits = self.bits & ~SymSet(other).bits
        return out

    def __and__(self, other: SymbolsLike) -> "SymSet":
        out = SymSet()
        out.bits = self.bits & SymSet(other).bits
        return out

    def __contains__(self, s: int) -> bool:
        return (self.bits >> int(s)) & 1 == 1

    def __bool__(self) -> bool:
        return self.bits != 0

    def __iter__(self):
        return (s for s in range(N_SYMBOLS) if (self.bits >> s) & 1)

    def __len__(self) -> int:
        return bin(self.bits).count("1")

    def __eq__(self, other) -> bool:
        return isinstance(other, SymSet) and other.bits == self.bits

    def __hash__(self) -> int:
        return hash(self.bits)

    def words(self) -> np.ndarray:
        return np.array([(self.bits >> (32 * i)) & 0xFFFFFFFF for i in range(SET_WORDS)],
                        dtype=np.uint32)


DIGITS = SymSet(b"0123456789")
ALL_BYTES = SymSet.all_bytes()


class Op:
    """Base class of the operator nodes."""


@dataclass
class Write(Op):
    literal: bytes

    def __post_init__(self):
        if isinstance(self.literal, str):
            self.literal = self.literal.encode("utf-8")


@dataclass
class Wait(Op):
    allow: SymSet
    wait: SymSet
    deny: SymSet = field(default_factory=SymSet)
    body: Optional[Op] = None

    def __post_init__(self):
        self.allow = SymSet(self.allow)
        self.wait = SymSet(self.wait)
        self.deny = SymSet(self.deny)


@dataclass
class WriteTokens(Op):
    """The paper's token-level Write: exactly these token ids, one per decode step."""

    tokens: List[int]


@dataclass
class Hole(Op):
    """The place of run-time argument ``arg`` in a template tree."""

    arg: int


@dataclass
class WaitUntil(Op):
    """A Wait whose wait "token" is a multi-byte string: text over ``allow`` (minus ``deny``)
    and the string's own bytes, up to and including the first occurrence of ``until``."""

    allow: SymSet
    until: bytes
    deny: SymSet = field(default_factory=SymSet)
    body: Optional[Op] = None

    def __post_init__(self):
        self.allow = SymSet(self.allow)
        self.deny = SymSet(self.deny)
        if isinstance(self.until, str):
            self.until = self.until.encode("utf-8")


@dataclass
class Cond:
    """The boolean Wait of an IfElse or DoWhile (true_waits / false_waits)."""

    allow: SymSet
    true_waits: SymSet
    false_waits: SymSet
    deny: SymSet = field(default_factory=SymSet)

    def __post_init__(self):
        self.allow = SymSet(self.allow)
        self.true_waits = SymSet(self.true_waits)
        self.false_waits = SymSet(self.false_waits)
        self.deny = SymSet(self.deny)


@dataclass
class Switch(Op):
    """k-way generalisation of IfElse: the deciding symbol picks the body."""

    allow: SymSet
    cases: List[SymSet]
    bodies: List[Optional[Op]]
    deny: SymSet = field(default_factory=SymSet)

    def __post_init__(self):
        self.allow = SymSet(self.allow)
        self.deny = SymSet(self.deny)
        self.cases = [SymSet(c) for c in self.cases]
        if len(self.cases) != len(self.bodies):
            raise ValueError("Switch needs one body per case")


def IfElse(condition: Cond, if_body: Optional[Op], else_body: Optional[Op]) -> Switch:
    return Switch(allow=condition.allow, deny=condition.deny,
                  cases=[condition.true_waits, condition.false_waits],
                  bodies=[if_body, else_body])


@dataclass
class DoWhile(Op):
    body: Optional[Op]
    condition: Cond


@dataclass
class Sequence(Op):
    parts: List[Op]

    def __init__(self, *parts: Op):
        if len(parts) == 1 and isinstance(parts[0], (list, tuple)):
            parts = tuple(parts[0])
        self.parts = list(parts)


@dataclass
class FlatTree:
    nodes: np.ndarray
    children: np.ndarray
    sets: np.ndarray
    data: np.ndarray
    root: int

    @property
    def n_nodes(self) -> int:
        return int(self.nodes.shape[0])


def flatten(root: Op) -> FlatTree:
    """Serialise a tree of operator objects into the flat arrays (pre-order)."""
    nodes: List[List[int]] = []
    children: List[int] = []
    sets: List[np.ndarray] = []
    data = bytearray()

    # iterative pre-order so that very deep enum tries do not hit the recursion limit
    def new_node(kind: int) -> int:
        nodes.append([kind, 0, 0, 0, 0, 0, 0, 0])
        return len(nodes) - 1

    def add_sets(idx: int, ss: Seq[SymSet]) -> None:
        nodes[idx][3] = len(ss)
        nodes[idx][4] = len(sets)
        for s in ss:
            sets.append(s.words())

    def reserve_children(idx: int, n: int) -> int:
        nodes[idx][1] = n
        nodes[idx][2] = len(children)
        children.extend([-1] * n)
        return nodes[idx][2]

    root_slot = [-1]
    # work items: (op, where to store the node index: (list, position))
    stack = [(root, root_slot, 0)]
    while stack:
        op, dest, pos = stack.pop()
        if op is None:
            dest[pos] = -1
            continue
        if isinstance(op, Write):
            idx = new_node(KIND_WRITE)
            nodes[idx][5] = len(data)
            nodes[idx][6] = len(op.literal)
            data.extend(op.literal)
            kids: List[Optional[Op]] = []
        elif isinstance(op, Wait):
            idx = new_node(KIND_WAIT)
            add_sets(idx, [op.allow, op.deny, op.wait])
            kids = [op.body]
        elif isinstance(op, WriteTokens):
            idx = new_node(KIND_WRITE_TOKENS)
            raw = np.asarray(op.tokens, dtype="<i4").tobytes()
            nodes[idx][5] = len(data)
            nodes[idx][6] = len(raw)
            data.extend(raw)
            kids = []
        elif isinstance(op, Hole):
            idx = new_node(KIND_HOLE)
            nodes[idx][7] = int(op.arg)
            kids = []
        elif isinstance(op, WaitUntil):
            idx = new_node(KIND_WAIT_UNTIL)
            add_sets(idx, [op.allow, op.deny])
            nodes[idx][5] = len(data)
            nodes[idx][6] = len(op.until)
            data.extend(op.until)
            kids = [op.body]
        elif isinstance(op, Switch):
            idx = new_node(KIND_SWITCH)
            add_sets(idx, [op.allow, op.deny] + list(op.cases))
            kids = list(op.bodies)
        elif isinstance(op, DoWhile):
            idx = new_node(KIND_DOWHILE)
            c = op.condition
            add_sets(idx, [c.allow, c.deny, c.true_waits, c.false_waits])
            kids = [op.body]
        elif isinstance(op, Sequence):
            idx = new_node(KIND_SEQUENCE)
            kids = list(op.parts)
        else:
            raise TypeError(f"not an operator: {op!r}")
        dest[pos] = idx
        if kids:
            off = reserve_children(idx, len(kids))
            for j in reversed(range(len(kids))):
                stack.append((kids[j], children, off + j))

    return FlatTree(
        nodes=np.asarray(nodes, dtype=np.int32).reshape(-1, 8),
        children=np.asarray(children, dtype=np.int32),
        sets=(np.stack(sets).astype(np.uint32) if sets else np.zeros((0, SET_WORDS), np.uint32)),
        data=np.frombuffer(bytes(data), dtype=np.uint8).copy(),
        root=int(root_slot[0]),
    )


def enum_trie(strings: Seq[bytes]) -> Op:
    """Operator tree accepting exactly one of ``strings`` (none a prefix of another).

    Each trie node with several continuations becomes a Switch whose cases are
    the single next bytes; single-continuation runs become Write literals.
    """
    strings = sorted(set(bytes(s) for s in strings))
    if not strings:
        raise ValueError("empty enum")
    for a, b in zip(strings, strings[1:]):
        if b.startswith(a):
            raise ValueError("enum strings must be prefix-free")

    def build(group: List[bytes], depth: int) -> Optional[Op]:
        # all strings in group share the first `depth` bytes
        if len(group) == 1:
            rest = group[0][depth:]
            return Write(rest) if rest else None
        # longest common prefix beyond depth
        lcp = depth
        first, last = group[0], group[-1]
        while lcp < len(first) and lcp < len(last) and first[lcp] == last[lcp]:
            lcp += 1
        by_byte: dict = {}
        for s in group:
            by_byte.setdefault(s[lcp], []).append(s)
        keys = sorted(by_byte)
        sw = Switch(allow=SymSet(keys), cases=[SymSet([k]) for k in keys],
                    bodies=[build(by_byte[k], lcp + 1) for k in keys])
        if lcp > depth:
            return Sequence(Write(first[depth:lcp]), sw)
        return sw

    out = build(strings, 0)
    assert out is not None
    return out


def substitute(op: Optional[Op], args: Seq[Optional[Op]]) -> Optional[Op]:
    """The tree with every ``Hole(i)`` replaced by ``args[i]`` (a fresh copy per occurrence)."""
    import copy
    if op is None:
        return None
    if isinstance(op, Hole):
        return copy.deepcopy(args[op.arg])
    if isinstance(op, Sequence):
        return Sequence([substitute(p, args) for p in op.parts])
    if isinstance(op, Switch):
        return Switch(allow=op.allow, cases=list(op.cases), deny=op.deny,
                      bodies=[substitute(b, args) for b in op.bodies])
    if isinstance(op, DoWhile):
        return DoWhile(body=substitute(op.body, args), condition=op.condition)
    if isinstance(op, Wait):
        return Wait(allow=op.allow, wait=op.wait, deny=op.deny, body=substitute(op.body, args))
    if isinstance(op, WaitUntil):
        return WaitUntil(allow=op.allow, until=op.until, deny=op.deny,
                         body=substitute(op.body, args))
    return op  # Write, WriteTokens: leaves without holes
