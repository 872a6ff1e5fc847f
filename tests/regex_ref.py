"""An independent statement of the operator languages as regular expressions.

Each operator's language (Write: the literal; Wait: stay* w body; Switch / IfElse:
stay* (s_i body_i); DoWhile: (body stay* t)* body stay* f; Sequence: concatenation) is
written as a pattern for the third-party ``regex`` module, whose backtracking matcher and
``partial=True`` mode (could this string be the beginning of a match?) share nothing with the
cursor interpreter under ``oracle/``.  The end-of-sequence symbol is carried as byte 0x02,
which never occurs in the generated vocabularies' token bytes.
"""
from __future__ import annotations

import regex

from wg_workloads.optree import EOS, DoWhile, Sequence, Switch, SymSet, Wait, WaitUntil, Write

EOS_BYTE = 0x02


def to_bytes(symbols) -> bytes:
    return bytes(EOS_BYTE if s == EOS else s for s in symbols)


def _cls(s: SymSet) -> bytes:
    members = []
    for sym in s:
        if sym == EOS:
            members.append(EOS_BYTE)
        elif sym != EOS_BYTE:
            members.append(sym)
    assert members, "empty symbol class"
    return b"[" + b"".join(b"\\x%02x" % m for m in sorted(set(members))) + b"]"


def _star(s: SymSet) -> bytes:
    real = [sym for sym in s if sym == EOS or sym != EOS_BYTE]
    return _cls(s) + b"*" if real else b""


def _union(sets) -> SymSet:
    out = SymSet()
    for s in sets:
        out = out | s
    return out


def pattern(op) -> bytes:
    if op is None:
        return b""
    if isinstance(op, Write):
        return b"".join(b"\\x%02x" % b for b in op.literal)
    if isinstance(op, Wait):
        stay = (op.allow - op.deny) - op.wait
        return _star(stay) + _cls(op.wait) + pattern(op.body)
    if isinstance(op, WaitUntil):
        # any accepted symbol as long as the string does not START here, then the string
        lit = b"".join(b"\\x%02x" % b for b in op.until)
        ok = (op.allow - op.deny) | SymSet(op.until)
        return b"(?:(?!" + lit + b")" + _cls(ok) + b")*" + lit + pattern(op.body)
    if isinstance(op, Switch):
        stay = (op.allow - op.deny) - _union(op.cases)
        alts = b"|".join(_cls(c) + pattern(b) for c, b in zip(op.cases, op.bodies))
        return _star(stay) + b"(?:" + alts + b")"
    if isinstance(op, DoWhile):
        c = op.condition
        stay = (c.allow - c.deny) - (c.true_waits | c.false_waits)
        body = pattern(op.body)
        return (b"(?:" + body + _star(stay) + _cls(c.true_waits) + b")*" + body + _star(stay)
                + _cls(c.false_waits))
    if isinstance(op, Sequence):
        return b"".join(pattern(p) for p in op.parts)
    raise TypeError(op)


def mentions_eos(op) -> bool:
    if op is None or isinstance(op, Write):
        return False
    if isinstance(op, Wait):
        return any(EOS in s for s in (op.allow, op.deny, op.wait)) or mentions_eos(op.body)
    if isinstance(op, WaitUntil):
        return EOS in op.allow or EOS in op.deny or mentions_eos(op.body)
    if isinstance(op, Switch):
        return (any(EOS in s for s in [op.allow, op.deny] + op.cases)
                or any(mentions_eos(b) for b in op.bodies))
    if isinstance(op, DoWhile):
        c = op.condition
        return (any(EOS in s for s in (c.allow, c.deny, c.true_waits, c.false_waits))
                or mentions_eos(op.body))
    return any(mentions_eos(p) for p in op.parts)


def program(op):
    """Compiled pattern of the whole program: the tree, the implicit EOS when no set
    mentions it, then any number of further EOS (a finished request only emits EOS)."""
    tail = b"" if mentions_eos(op) else b"\\x02"
    return regex.compile(b"(?s)" + pattern(op) + tail + b"\\x02*")


def viable(prog, data: bytes) -> bool:
    return prog.fullmatch(data, partial=True) is not None


def member(prog, data: bytes) -> bool:
    m = prog.fullmatch(data)
    return m is not None
