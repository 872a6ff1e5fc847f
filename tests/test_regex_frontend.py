"""The regular-expression front end (paper Section 3.2: regex -> Wait / Write / IfElse /
DoWhile compositions) pinned against the standard library's ``re``: for every pattern, every
string over a small alphabet up to a length bound must be accepted by the generated operator
tree (interpreted by the CPU checker) and by the compiled table exactly when ``re.fullmatch``
accepts it."""
import itertools
import re

import pytest

import oracle
from wg_workloads import EOS
from wg_workloads.optree import FlatTree


@pytest.fixture(scope="module")
def wg():
    from paper_2507_16768_b200 import build
    build.build()
    import paper_2507_16768_b200 as wg
    return wg


CASES = [
    (r"\d+(\.\d+)*", "07.x", 7),                       # the paper's worked example
    (r"abc", "abcx", 5),
    (r"[a-c]+x", "abcx", 6),
    (r"a*b", "abx", 6),
    (r"a*b*c", "abcx", 6),
    (r"(ab)*c", "abcx", 7),
    (r"(ab)+c", "abcx", 7),
    (r"x(,\d+)*;", "x,0;7", 8),
    (r"(a|bc|d)e", "abcde", 5),
    (r"(a|b)*c", "abcx", 6),
    (r"(a\d*|b)c", "ab0c7", 6),
    (r"ab?c", "abcx", 5),
    (r"(ab)?c", "abcx", 5),
    (r"a(b|c)?d", "abcd", 5),
    (r"\[\d+(,\d+)*\]", "[],07", 8),
    (r'"[^"]*"', '"ab\\', 6),
    (r"a{2,4}b", "abx", 7),
    (r"(ab){2}c", "abc", 7),
    (r"a{2,}b", "abx", 7),
    (r"[0-9a-f]{2}(:[0-9a-f]{2})*", "0a:f.", 8),
    (r"(true|false|null)", "truefalsn", 5),
    (r"-?\d+", "-07x", 5),
    (r"\w+@\w+\.com", "a@.com", 7),
    (r"^ab$", "ab^$", 4),
    (r"\x41\n\t", "A\n\tx", 4),
    (r"", "a", 2),
    (r"a.c", "a\nbc", 4),
]


def enumerate_strings(alphabet, max_len):
    for n in range(max_len + 1):
        for tup in itertools.product(alphabet, repeat=n):
            yield "".join(tup)


@pytest.mark.parametrize("pattern,alphabet,max_len", CASES)
def test_regex_language_equals_stdlib_re(wg, pattern, alphabet, max_len):
    tree_arrays = wg.binding.RegexTree(pattern)
    flat = FlatTree(tree_arrays.nodes, tree_arrays.children, tree_arrays.sets, tree_arrays.data,
                    tree_arrays.root)
    tree = oracle.Tree(flat)
    g = wg.Grammar.from_regex(pattern)
    g2 = wg.Grammar(flat)
    assert g.content_hash == g2.content_hash
    want = re.compile(pattern.encode(), re.S if False else 0)
    syms = sorted(set(alphabet.encode()))
    n_members = 0

    # walk both automata over the prefix tree of all strings, so every string is checked once
    def dfs(cursor, sid, text, depth):
        nonlocal n_members
        member = want.fullmatch(text) is not None
        end_c = tree.step(cursor, EOS) if not oracle.is_dead(cursor) else cursor
        accepted_tree = end_c == oracle.DONE
        accepted_table = sid != 0 and g.step(sid, EOS) == g.done_state
        assert accepted_tree == member, (pattern, text)
        assert accepted_table == member, (pattern, text)
        n_members += member
        if depth == max_len:
            return
        for s in syms:
            nxt = tree.step(cursor, s) if not oracle.is_dead(cursor) else cursor
            nsid = g.step(sid, s) if sid else 0
            assert oracle.is_dead(nxt) == (nsid == 0)
            if nsid == 0:
                # a refused prefix must have no accepted extension within the bound
                if depth + 1 <= 3:
                    for tail in enumerate_strings(alphabet, min(2, max_len - depth - 1)):
                        assert want.fullmatch(text + bytes([s]) + tail.encode()) is None
                continue
            dfs(nxt, nsid, text + bytes([s]), depth + 1)

    dfs(tree.start(), g.start_state, b"", 0)
    if pattern not in ("",):
        assert n_members >= 1


def test_paper_example_has_the_shape_of_the_listing(wg):
    from paper_2507_16768_b200.binding import RegexTree
    t = RegexTree(r"\d+(\.\d+)*")
    kinds = t.nodes[:, 0].tolist()
    # Sequence(Wait one digit, Switch(EOS -> nothing, '.' -> DoWhile(Wait one digit, cond)))
    assert kinds == [0, 2, 3, 4, 2]
    switch = t.nodes[2]
    assert switch[1] == 2 and switch[3] == 4            # two cases, allow + deny + 2 case sets
    assert t.children[switch[2]] == -1                   # the EOS case has no body


@pytest.mark.parametrize("pattern,why", [
    (r"a*a", "runs into"),
    (r"(a|ab)c", "same symbol"),
    (r"(ab)*a", "same symbol"),
    (r"\d+\d", "runs into"),
    (r"a*b*c*d", "separator"),
    (r"(a*)*b", "at least one symbol"),
    (r"(", "missing"),
    (r"a)", "unbalanced"),
    (r"[abc", "unterminated"),
    (r"*a", "unexpected"),
    (r"\q", "unsupported escape"),
    (r"(?=a)b", "unsupported group"),
    (r"x{5,2}", "bad"),
])
def test_patterns_outside_the_dialect_are_refused_with_a_reason(wg, pattern, why):
    with pytest.raises(wg.WgError) as e:
        wg.Grammar.from_regex(pattern)
    assert e.value.status == wg.binding.WG_ERR_GRAMMAR
    assert why in str(e.value), str(e.value)


def test_golden_fixture_through_the_regex_front_end(wg):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "section_3_2_listing_language.txt")
    g = wg.Grammar.from_regex(r"\d+(\.\d+)*")
    for line in open(path):
        line = line.rstrip("\n")
        if not line or line.startswith("#"):
            continue
        verdict, text = line.split(" ", 1)
        text = "" if text == "<empty>" else text
        end = g.walk(g.start_state, [ord(c) for c in text] + [EOS])
        assert (end == g.done_state) is (verdict == "accept"), line
