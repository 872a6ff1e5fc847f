"""Seeded operator-tree generators for the five workloads.

The trees only take the *shape* of the paper's tasks (Section 1: an HTML-like
outline with fixed tags in a fixed order and free text between them; a JSON
array of objects with fixed keys, a topic index and id-path strings).  None of
the paper's datasets is reproduced.
"""
from __future__ import annotations

from typing import List

import numpy as np

from .optree import (ALL_BYTES, DIGITS, Cond, DoWhile, Hole, IfElse, Op, Sequence, Switch, SymSet,
                     Wait, WaitUntil, Write, enum_trie, substitute)

LT = ord("<")


def dotted_number() -> Op:
    """One or more digits, then any number of groups of a period and one or more digits, then the
    end of sequence: the language Section 3.2 states for its worked example, built here from that
    statement (a digit, then "more digits or a period and a digit again" as a loop)."""
    from .optree import EOS
    digit = Wait(allow=DIGITS, wait=DIGITS)
    return DoWhile(body=digit,
                   condition=Cond(allow=DIGITS | b"." | [EOS], true_waits=SymSet(b"."),
                                  false_waits=SymSet([EOS])))


def text_slot(closing: bytes) -> List[Op]:
    """Free text up to the first '<', then the rest of the closing tag."""
    assert closing[:1] == b"<"
    return [Wait(allow=ALL_BYTES, wait=SymSet([LT])), Write(closing[1:])]


HTML_TAGS = [
    (b'<h1 class="document-title" id="outline-root">', b"</h1>\n"),
    (b'<p class="document-abstract" data-level="0">', b"</p>\n"),
    (b'<h2 class="section-title" id="outline-section-1">', b"</h2>\n"),
    (b'<p class="section-summary" data-level="1">', b"</p>\n"),
]


def html_template(wait_for_tag: bool = False) -> Op:
    """Config 1: eight literal tags in a fixed order with four free-text slots.

    By default a slot is free of '<' and ends at the first '<' (single-symbol wait sets).
    With ``wait_for_tag`` the slot is a Wait on the whole closing tag: any text, '<' included,
    up to the first occurrence of the tag.
    """
    parts: List[Op] = []
    for open_tag, close_tag in HTML_TAGS:
        parts.append(Write(open_tag))
        if wait_for_tag:
            parts.append(WaitUntil(ALL_BYTES, close_tag))
        else:
            parts.extend(text_slot(close_tag))
    return Sequence(parts)


def int_0_63(terminator: bytes) -> Op:
    """Decimal 0..63 without leading zeros, ended by ``terminator`` (one byte)."""
    term = SymSet(terminator)
    end = Write(terminator)
    return Switch(
        allow=DIGITS,
        cases=[SymSet(b"0789"), SymSet(b"12345"), SymSet(b"6")],
        bodies=[
            end,
            Switch(allow=DIGITS | term, cases=[DIGITS, term], bodies=[Write(terminator), None]),
            Switch(allow=SymSet(b"0123") | term, cases=[SymSet(b"0123"), term],
                   bodies=[Write(terminator), None]),
        ],
    )


def id_path_string() -> Op:
    """A quoted string of /-separated decimal node ids (``"12/7/3"``): the language of
    ``dotted_number`` with '/' for the period and a closing quote for the end of sequence."""
    digit = Wait(allow=DIGITS, wait=DIGITS)
    return Sequence(
        Write(b'"'),
        DoWhile(body=digit,
                condition=Cond(allow=DIGITS | b'/"', true_waits=SymSet(b"/"),
                               false_waits=SymSet(b'"'))),
    )


def document_node_paths(seed: int, n_nodes: int) -> List[bytes]:
    """Node-id paths ("3", "3/1", "3/1/12", ...) of a seeded random document tree."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x646F63]))
    paths: List[bytes] = []
    frontier: List[tuple] = [(b"", 0)]
    while frontier and len(paths) < n_nodes:
        prefix, depth = frontier.pop(int(rng.integers(0, len(frontier))))
        fan = int(rng.integers(2, 16)) if depth < 4 else 0
        for k in range(1, fan + 1):
            if len(paths) >= n_nodes:
                break
            path = (prefix + b"/" if prefix else b"") + str(k).encode()
            paths.append(path)
            frontier.append((path, depth + 1))
    return paths


def json_reference_lookup(doc_seed: int = 0, doc_nodes: int = 1350) -> Op:
    """Configs 2 and 4: an array of {"topic": <0..63>, "paths": [<id path>, ...]}.

    With ``doc_nodes`` > 0 every path string must be the id path of a node of the request's
    document (Section 1: values are restricted to section ids), an enum over a seeded random
    document tree; with ``doc_nodes`` = 0 it is any /-separated run of decimal ids.
    """
    more_or_close = Cond(allow=SymSet(b",]"), true_waits=SymSet(b","), false_waits=SymSet(b"]"))
    if doc_nodes > 0:
        names = [p + b'"' for p in document_node_paths(doc_seed, doc_nodes)]
        path = Sequence(Write(b'"'), enum_trie(names))
    else:
        path = id_path_string()
    obj = Sequence(
        Write(b'{"topic": '),
        int_0_63(b","),
        Write(b' "paths": ['),
        DoWhile(body=path, condition=more_or_close),
        Write(b"}"),
    )
    return Sequence(Write(b"["), DoWhile(body=obj, condition=more_or_close))


PRINTABLE = np.frombuffer(
    b"abcdefghijklmnopqrstuvwxyzABCDEFGHIJKLMNOPQRSTUVWXYZ0123456789 _-.:=/\"'<>{}[](),;",
    dtype=np.uint8)


def _literal(rng: np.random.Generator, lo: int, hi: int) -> bytes:
    n = int(rng.integers(lo, hi + 1))
    return PRINTABLE[rng.integers(0, PRINTABLE.size, size=n)].tobytes()


def random_template(seed: int, min_segments: int = 10, max_segments: int = 30) -> Op:
    """Config 3: literal segments of 2..12 bytes with a Wait / IfElse / DoWhile slot between."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x74656D706C]))
    n_seg = int(rng.integers(min_segments, max_segments + 1))
    parts: List[Op] = []
    for i in range(n_seg):
        parts.append(Write(_literal(rng, 2, 12)))
        if i == n_seg - 1:
            break
        kind = int(rng.integers(0, 3))
        if kind == 0:
            stop = int(rng.choice(np.frombuffer(b"<>\"};|", dtype=np.uint8)))
            parts.append(Wait(allow=ALL_BYTES, wait=SymSet([stop])))
        elif kind == 1:
            a, b = (int(x) for x in rng.choice(np.frombuffer(b"01ynTF+-", dtype=np.uint8),
                                               size=2, replace=False))
            parts.append(IfElse(
                condition=Cond(allow=SymSet([a, b]), true_waits=SymSet([a]),
                               false_waits=SymSet([b])),
                if_body=Write(_literal(rng, 12, 48)),
                else_body=(Write(_literal(rng, 12, 48)) if rng.random() < 0.7 else None)))
        else:
            sep, end = (int(x) for x in rng.choice(np.frombuffer(b",;|]})", dtype=np.uint8),
                                                  size=2, replace=False))
            item = Sequence(Write(_literal(rng, 8, 32)), Wait(allow=DIGITS, wait=DIGITS))
            parts.append(DoWhile(
                body=item,
                condition=Cond(allow=DIGITS | [sep, end], true_waits=SymSet([sep]),
                               false_waits=SymSet([end]))))
    return Sequence(parts)


ENUM_ALPHABET = np.frombuffer(b"abcdefghijklmnopqrstuvwxyz0123456789-_", dtype=np.uint8)


def dynamic_snippet_parts(seed: int, n_args: int = 64, enum_size: int = 40,
                          len_min: int = 3, len_max: int = 12):
    """Config 5 as (template, arguments): the static HTML structure with one hole per section
    (Section 3.1: parameterised, not yet instantiated) and the per-request enums that fill them.

    Section ``i`` is ``<sec name="`` + one of ``enum_size`` random strings + ``">`` + free text +
    ``</sec>``.  Each enum is a trie of k-way Switch nodes; the closing quote is part of every
    string so that no entry is a prefix of another.  The static part does not depend on the seed.
    """
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x736E6970]))
    parts: List[Op] = []
    args: List[Op] = []
    for i in range(n_args):
        names = set()
        while len(names) < enum_size:
            n = int(rng.integers(len_min, len_max + 1))
            names.add(ENUM_ALPHABET[rng.integers(0, ENUM_ALPHABET.size, size=n)].tobytes() + b'"')
        parts.append(Write(b'<sec name="'))
        parts.append(Hole(i))
        args.append(enum_trie(sorted(names)))
        parts.append(Write(b">"))
        parts.extend(text_slot(b"</sec>\n"))
    return Sequence(parts), args


def dynamic_snippet_template(seed: int, n_args: int = 64, enum_size: int = 40,
                             len_min: int = 3, len_max: int = 12) -> Op:
    """Config 5 as one tree: ``dynamic_snippet_parts`` with the arguments filled in."""
    template, args = dynamic_snippet_parts(seed, n_args, enum_size, len_min, len_max)
    return substitute(template, args)
