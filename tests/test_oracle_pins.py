"""Pins of the CPU checker against things other than itself.

* the paper's worked example (Section 3.2 listing) against a hand-written standard-library
  regular expression of the pattern the paper says it represents;
* the non-greedy rule (Section 6);
* masks against an independent partial matcher (``regex_ref``) and against brute-force
  prefix viability on tiny vocabularies;
* closed forms: single-byte tokens, pure literals, one free-text slot;
* the invariants the method promises: the EOS rule, non-empty masks on a valid trajectory,
  the decoded trajectory being a member of the language;
* apply / argmax against their plain definitions in numpy.
"""
import itertools
import re

import numpy as np
import pytest

import oracle
import regex_ref
from wg_workloads import (ALL_BYTES, DIGITS, EOS, Cond, DoWhile, IfElse, Sequence, Switch, SymSet,
                          Wait, WaitUntil, Write, WriteTokens, bf16_bits_to_f32, enum_trie, flatten, grammars,
                          make_logits, make_vocab, vocab_from_tokens)


def tree_of(op):
    return oracle.Tree(flatten(op))


def bit(words, t):
    return (int(words[t >> 5]) >> (t & 31)) & 1


def unpack(words, V):
    return np.unpackbits(words.view(np.uint8), bitorder="little")[:V].astype(bool)


# ---------------------------------------------------------------------------------------
# Section 3.2, worked example: an operator tree said to represent \d+(\.\d+)* followed by <eos>
# ---------------------------------------------------------------------------------------
def worked_example_tree():
    """The example's operator tree, read from its fixture (tests/golden)."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "section_3_2_worked_example_tree.txt")
    text = " ".join(l for l in open(path).read().splitlines() if not l.startswith("#"))
    tokens = text.replace("(", " ( ").replace(")", " ) ").split()
    named = {"digits": SymSet(b"0123456789"), "dot": SymSet(b"."), "eos": SymSet([EOS])}

    def symset(spec):
        out = SymSet()
        for name in spec.split("+"):
            out = out | named[name]
        return out

    def parse(i):
        assert tokens[i] == "("
        kind, i = tokens[i + 1], i + 2
        sets, kids = {}, []
        while tokens[i] != ")":
            if tokens[i] == "(":
                kid, i = parse(i)
                kids.append(kid)
            else:
                key, spec = tokens[i].split("=")
                sets[key] = symset(spec)
                i += 1
        if kind == "none":
            return None, i + 1
        if kind == "sequence":
            return Sequence(kids), i + 1
        if kind == "wait":
            return Wait(allow=sets["allow"], wait=sets["wait"]), i + 1
        cond = Cond(allow=sets["allow"], true_waits=sets["true"], false_waits=sets["false"])
        if kind == "ifelse":
            return IfElse(condition=cond, if_body=kids[0], else_body=kids[1]), i + 1
        assert kind == "dowhile"
        return DoWhile(body=kids[0], condition=cond), i + 1

    return parse(0)[0]


@pytest.mark.parametrize("which", ["worked example", "dotted_number"])
def test_paper_listing_language_exhaustive(which):
    # the paper's own tree, and the tree the workloads build from the stated language
    tree = tree_of(worked_example_tree() if which == "worked example" else grammars.dotted_number())
    hand = re.compile(rb"[0-9]+(\.[0-9]+)*\x02+")
    alphabet = [ord("0"), ord("7"), ord("."), ord("x"), EOS]
    n_accept = 0

    def dfs(cursor, symbols):
        nonlocal n_accept
        data = regex_ref.to_bytes(symbols)
        accepted = cursor == oracle.DONE
        assert accepted == (hand.fullmatch(data) is not None), data
        n_accept += accepted
        if len(symbols) == 7:
            return
        for s in alphabet:
            nxt = tree.step(cursor, s)
            if oracle.is_dead(nxt):
                # everything below a refused symbol must be a non-member as well
                assert hand.fullmatch(regex_ref.to_bytes(symbols + [s])) is None
                if len(symbols) < 5:
                    for tail in itertools.product(alphabet, repeat=2):
                        assert hand.fullmatch(regex_ref.to_bytes(symbols + [s] + list(tail))) is None
                continue
            dfs(nxt, symbols + [s])

    dfs(tree.start(), [])
    assert n_accept > 100


def test_paper_listing_keeps_digit_runs_and_needs_a_digit_after_the_dot():
    tree = tree_of(worked_example_tree())
    ok = lambda s: tree.accepts([ord(c) for c in s] + [EOS])  # noqa: E731
    assert ok("7") and ok("2025") and ok("3.14") and ok("10.0.0.255")
    assert not ok("") and not ok(".5") and not ok("5.") and not ok("1..2") and not ok("1.x")
    # without the end-of-sequence symbol the program has not completed
    assert not tree.accepts([ord("7")])


def test_non_greedy_wait_ends_at_first_wait_symbol():
    tree = tree_of(Sequence(Wait(allow=SymSet(b"ab"), wait=SymSet(b"b")), Write(b"c")))
    assert tree.accepts(list(b"aabc") + [EOS])
    assert tree.accepts(list(b"bc") + [EOS])
    assert not tree.accepts(list(b"abbc") + [EOS])
    assert not tree.accepts(list(b"aac") + [EOS])


def test_wait_symbol_outside_allow_is_still_accepted_and_deny_wins_over_allow():
    tree = tree_of(Wait(allow=SymSet(b"abc"), deny=SymSet(b"c"), wait=SymSet(b";")))
    assert tree.accepts(list(b"abab;") + [EOS])
    assert not tree.accepts(list(b"abc;") + [EOS])


def test_wait_body_runs_after_the_wait_symbol():
    tree = tree_of(Sequence(Wait(allow=SymSet(b"x"), wait=SymSet(b"("), body=Write(b"in")),
                            Write(b")")))
    assert tree.accepts(list(b"xx(in)") + [EOS])
    assert not tree.accepts(list(b"xx()") + [EOS])


def test_switch_three_way_and_absent_bodies():
    sw = Switch(allow=SymSet(b" abc"), cases=[SymSet(b"a"), SymSet(b"b"), SymSet(b"c")],
                bodies=[Write(b"1"), None, Sequence(Write(b"3"), Write(b"3"))])
    tree = tree_of(Sequence(sw, Write(b".")))
    for s, want in [(b"a1.", True), (b"  b.", True), (b"c33.", True), (b"a.", False),
                    (b"b1.", False), (b"c3.", False), (b"d.", False)]:
        assert tree.accepts(list(s) + [EOS]) is want, s


def test_dowhile_repeats_on_true_and_leaves_on_false():
    loop = DoWhile(body=Write(b"ab"), condition=Cond(allow=SymSet(b" ,;"), true_waits=SymSet(b","),
                                                     false_waits=SymSet(b";")))
    tree = tree_of(Sequence(Write(b"["), loop, Write(b"]")))
    for s, want in [(b"[ab;]", True), (b"[ab,ab;]", True), (b"[ab ,ab  ;]", True),
                    (b"[;]", False), (b"[ab,;]", False), (b"[ab,ab]", False), (b"[abab;]", False)]:
        assert tree.accepts(list(s) + [EOS]) is want, s


def test_done_accepts_only_eos_and_stays_done():
    tree = tree_of(Write(b"hi"))
    c = tree.walk(tree.start(), list(b"hi"))
    assert c == (-3, 0)                        # the implicit trailing EOS wait
    assert oracle.is_dead(tree.step(c, ord("x")))
    c = tree.step(c, EOS)
    assert c == oracle.DONE
    assert tree.step(c, EOS) == oracle.DONE
    assert oracle.is_dead(tree.step(c, ord("h")))


def test_explicit_eos_suppresses_the_implicit_one():
    tree = tree_of(Sequence(Write(b"a"), Wait(allow=SymSet([EOS]), wait=SymSet([EOS]))))
    assert tree.walk(tree.start(), [ord("a"), EOS]) == oracle.DONE


@pytest.mark.parametrize("bad", [
    Wait(allow=SymSet(b"a"), wait=SymSet()),                                   # empty wait set
    Wait(allow=SymSet(b"ab"), wait=SymSet(b"b"), deny=SymSet(b"b")),           # wait meets deny
    IfElse(Cond(allow=SymSet(b"ab"), true_waits=SymSet(b"ab"), false_waits=SymSet(b"b")),
           None, None),                                                         # overlapping cases
    DoWhile(Write(b"x"), Cond(allow=SymSet(b"a"), true_waits=SymSet(b"a"), false_waits=SymSet())),
])
def test_rejected_trees(bad):
    with pytest.raises(oracle.OracleError) as e:
        tree_of(bad)
    assert e.value.code == oracle.ERR_GRAMMAR


def test_shared_subtree_is_rejected():
    flat = flatten(Sequence(Write(b"a"), Write(b"b")))
    flat.children[1] = flat.children[0]        # both parts point at the same node
    with pytest.raises(oracle.OracleError):
        oracle.Tree(flat)


# ---------------------------------------------------------------------------------------
# masks against the independent partial matcher
# ---------------------------------------------------------------------------------------
SMALL_GRAMMARS = {
    "dotted_number": grammars.dotted_number,
    "html": grammars.html_template,
    "json": grammars.json_reference_lookup,
    "template0": lambda: grammars.random_template(0, 4, 6),
    "template5": lambda: grammars.random_template(5, 4, 6),
    "snippets": lambda: grammars.dynamic_snippet_template(3, n_args=2, enum_size=7),
    "html_tags": lambda: grammars.html_template(wait_for_tag=True),
}


def greedy_random_walk(tree, vocab, rng, steps, prefer=None):
    """Yield (cursor, emitted symbols so far) along a random valid trajectory."""
    cursor, emitted = tree.start(), []
    for _ in range(steps):
        yield cursor, list(emitted)
        allowed = np.flatnonzero(unpack(oracle.mask(tree, vocab, cursor), vocab.size))
        assert allowed.size > 0
        pool = allowed
        if prefer is not None and rng.random() < 0.7:
            good = allowed[prefer[allowed]]
            if good.size:
                pool = good
        t = int(rng.choice(pool))
        rc, cursor = oracle.advance(tree, vocab, cursor, t)
        assert rc == 0
        emitted += [EOS] if t == vocab.eos_id else list(vocab.token(t))


@pytest.mark.parametrize("name", sorted(SMALL_GRAMMARS))
def test_masks_equal_partial_regex_matching(name):
    from wg_workloads import has_structural_byte
    op = SMALL_GRAMMARS[name]()
    tree = tree_of(op)
    prog = regex_ref.program(op)
    vocab = make_vocab(1500, seed=11)
    toks = vocab.tokens()
    rng = np.random.default_rng(7)
    prefer = has_structural_byte(vocab)
    n_points = 0
    for cursor, emitted in greedy_random_walk(tree, vocab, rng, 40, prefer):
        prefix = regex_ref.to_bytes(emitted)
        got = unpack(oracle.mask(tree, vocab, cursor), vocab.size)
        for t in range(vocab.size):
            if t == vocab.eos_id:
                want = regex_ref.viable(prog, prefix + bytes([regex_ref.EOS_BYTE]))
            elif len(toks[t]) == 0:
                want = False
            else:
                want = regex_ref.viable(prog, prefix + toks[t])
            assert bool(got[t]) == want, (name, t, toks[t], prefix[-20:])
        n_points += 1
    assert n_points == 40


def test_mask_is_prefix_viability_by_brute_force_on_a_tiny_vocabulary():
    # [TEXT</] with TEXT free of '<'; membership decided by a hand-written stdlib pattern
    op = Sequence(Write(b"["), Wait(allow=ALL_BYTES, wait=SymSet(b"<")), Write(b"/]"))
    hand = re.compile(rb"\[[^<\x02]*</\]\x02+", re.S)
    tree = tree_of(op)
    alphabet = [b"<", b"[", b"]", b"/", b"x", b"\x02"]
    tokens = [b"<", b"[", b"", b"]", b"/", b"x", b"[<", b"/]", b"[x", b"x<", b"</", b"</]",
              b"xx", b"<<", b"[</]", b"]x</", b"</]x", b"[[", b"x]/", b"[x</]", b"/]x", b"<]"]
    vocab = vocab_from_tokens(tokens, eos_id=2)

    def viable(data):
        for n in range(0, 7):
            for z in itertools.product(alphabet, repeat=n):
                if hand.fullmatch(data + b"".join(z)):
                    return True
        return False

    prefixes = [b"", b"[", b"[x", b"[x]x/", b"[<", b"[xx<", b"[x</", b"[x</]"]
    for p in prefixes:
        cursor = tree.walk(tree.start(), list(p))
        assert not oracle.is_dead(cursor)
        got = unpack(oracle.mask(tree, vocab, cursor), vocab.size)
        for t, tok in enumerate(tokens):
            data = p + (b"\x02" if t == 2 else tok)
            want = False if (t != 2 and not tok) else viable(data)
            assert bool(got[t]) == want, (p, tok)


# ---------------------------------------------------------------------------------------
# closed forms on the config-1 vocabulary
# ---------------------------------------------------------------------------------------
@pytest.fixture(scope="module")
def vocab32k():
    return make_vocab(32000, seed=1)


def test_bit_order_and_zero_tail():
    tokens = [bytes([65 + (i % 26)]) * (1 + i // 26) for i in range(70)]
    tokens[2] = b""
    vocab = vocab_from_tokens(tokens, eos_id=2)
    tree = tree_of(Write(b"HH"))              # allowed: "H" (id 7) and "HH" (id 33)
    words = oracle.mask(tree, vocab, tree.start())
    assert words.shape == (3,)
    assert words.tolist() == [1 << 7, 1 << (33 - 32), 0]
    every = tree_of(Wait(allow=ALL_BYTES, wait=SymSet(b"!")))
    words = oracle.mask(every, vocab, every.start())
    assert words.tolist() == [0xFFFFFFFF & ~(1 << 2), 0xFFFFFFFF, (1 << 6) - 1]  # ids 64..69 only


def test_single_byte_tokens_follow_the_active_primitive(vocab32k):
    op = grammars.json_reference_lookup()
    tree = tree_of(op)
    prog = regex_ref.program(op)
    prefix = b'[{"topic": 1'
    cursor = tree.walk(tree.start(), list(prefix))
    words = oracle.mask(tree, vocab32k, cursor)
    for t in range(256):
        want = t != 2 and (chr(t) in "0123456789,")
        assert bit(words, t) == int(want), t
    assert regex_ref.viable(prog, prefix + b",")


def test_pure_literal_allows_exactly_the_prefixes_of_the_rest(vocab32k):
    lit = b'he said: "<p>ok</p>", twice'
    tree = tree_of(Write(lit))
    toks = vocab32k.tokens()
    for done in (0, 3, 10, len(lit) - 2):
        cursor = tree.walk(tree.start(), list(lit[:done]))
        got = unpack(oracle.mask(tree, vocab32k, cursor), vocab32k.size)
        rest = lit[done:]
        want = np.array([len(t) > 0 and rest.startswith(t) for t in toks])
        assert (got == want).all()
        assert got.sum() >= 1


def test_free_text_slot_closed_form(vocab32k):
    closing = b"/h1>"
    op = Sequence(Write(b"<h1>"), Wait(allow=ALL_BYTES, wait=SymSet(b"<")), Write(closing),
                  Write(b"<p>"))
    tree = tree_of(op)
    cursor = tree.walk(tree.start(), list(b"<h1>some text"))
    got = unpack(oracle.mask(tree, vocab32k, cursor), vocab32k.size)
    after = closing + b"<p>"
    for t, tok in enumerate(vocab32k.tokens()):
        if t == 2 or not tok:
            want = False
        elif b"<" not in tok:
            want = True
        else:
            want = after.startswith(tok[tok.index(b"<") + 1:])
        assert bool(got[t]) == want, tok
    assert 0.5 < got.mean() < 1.0


# ---------------------------------------------------------------------------------------
# invariants along decoded trajectories
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["html", "json", "template0", "snippets"])
def test_trajectory_invariants(name):
    from wg_workloads import has_structural_byte
    op = SMALL_GRAMMARS[name]()
    tree = tree_of(op)
    prog = regex_ref.program(op)
    vocab = make_vocab(4000, seed=3)
    bonus = has_structural_byte(vocab)
    cursor, emitted, finished = tree.start(), [], False
    for step in range(400):
        words = oracle.mask(tree, vocab, cursor)
        assert words.any(), "empty mask on a valid trajectory"
        # EOS rule: the EOS bit is set iff the EOS symbol is accepted here
        assert bit(words, vocab.eos_id) == int(not oracle.is_dead(tree.step(cursor, EOS)))
        logits = make_logits(1, vocab.size, "fp32", [99, 0], step, bonus, steer=6.0)
        t = int(oracle.argmax(logits, words[None, :], vocab.size)[0])
        assert bit(words, t) == 1
        rc, cursor = oracle.advance(tree, vocab, cursor, t)
        assert rc == 0
        emitted += [EOS] if t == vocab.eos_id else list(vocab.token(t))
        assert regex_ref.viable(prog, regex_ref.to_bytes(emitted))
        if cursor == oracle.DONE:
            finished = True
            break
    if finished:
        assert regex_ref.member(prog, regex_ref.to_bytes(emitted))
        # a finished request can only emit EOS
        words = oracle.mask(tree, vocab, cursor)
        assert unpack(words, vocab.size).sum() == 1 and bit(words, vocab.eos_id) == 1
    if name in ("json", "html"):
        assert finished, "steered greedy decoding should finish these templates"


def test_advance_rejects_and_keeps_the_cursor(vocab32k):
    tree = tree_of(Write(b"abc"))
    start = tree.start()
    rc, c = oracle.advance(tree, vocab32k, start, ord("b"))
    assert rc == oracle.ERR_REJECTED and c == start
    rc, c = oracle.advance(tree, vocab32k, start, vocab32k.size)
    assert rc == oracle.ERR_REJECTED and c == start
    rc, c = oracle.advance(tree, vocab32k, start, ord("a"))
    assert rc == 0 and c == (0, 1)


# ---------------------------------------------------------------------------------------
# apply and argmax against their definitions
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_apply_matches_numpy_definition(dtype):
    V, B = 1003, 5
    rng = np.random.default_rng(5)
    logits = make_logits(B, V, dtype, 1)
    words = rng.integers(0, 1 << 32, size=(B, (V + 31) // 32), dtype=np.uint64).astype(np.uint32)
    words[0] = 0xFFFFFFFF
    words[1] = 0
    keep = np.stack([unpack(words[r], V) for r in range(B)])
    before = logits.copy()
    oracle.apply_mask(logits, words, V)
    raw = logits.view(np.uint32) if dtype == "fp32" else logits
    raw_before = before.view(np.uint32) if dtype == "fp32" else before
    ninf = 0xFF800000 if dtype == "fp32" else 0xFF80
    assert (raw[keep] == raw_before[keep]).all()
    assert (raw[~keep] == ninf).all()
    assert (raw[0] == raw_before[0]).all() and (raw[1] == ninf).all()
    as_float = logits if dtype == "fp32" else bf16_bits_to_f32(logits)
    assert np.isneginf(as_float[~keep]).all()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_argmax_is_first_maximum_over_allowed(dtype):
    V, B = 5000, 6
    rng = np.random.default_rng(9)
    logits = make_logits(B, V, dtype, 2)
    words = rng.integers(0, 1 << 32, size=(B, (V + 31) // 32), dtype=np.uint64).astype(np.uint32)
    words[5] = 0
    got = oracle.argmax(logits, words, V)
    vals = logits if dtype == "fp32" else bf16_bits_to_f32(logits)
    for r in range(B - 1):
        keep = unpack(words[r], V)
        masked = np.where(keep, vals[r], -np.inf)
        assert got[r] == int(np.argmax(masked))     # numpy returns the first maximum
    assert got[5] == -1


def test_argmax_ties_signed_zero_and_all_minus_inf():
    V = 64
    words = np.array([[0xFFFFFFF0, 0xFFFFFFFF]], np.uint32)     # ids 0..3 are masked out
    x = np.full((1, V), -1.0, np.float32)
    x[0, 2] = 9.0                     # masked: must not win
    x[0, 10] = -0.0
    x[0, 20] = 0.0                    # equal to -0.0: the lower id stays
    assert oracle.argmax(x, words, V)[0] == 10
    x[0, 30] = 0.5
    x[0, 40] = 0.5
    assert oracle.argmax(x, words, V)[0] == 30
    x[:] = -np.inf
    assert oracle.argmax(x, words, V)[0] == 4
    bf = np.full((1, V), 0xBF80, np.uint16)                    # -1.0
    bf[0, 50] = 0x3F80                                          # +1.0
    bf[0, 60] = 0x3F80
    assert oracle.argmax(bf, words, V)[0] == 50


# ---------------------------------------------------------------------------------------
# adaptive allows / denies storage (Section 3.3) and the apply that works from such a set
# ---------------------------------------------------------------------------------------
def test_adaptive_token_set_hand_examples():
    # V = 10, allowed = {1, 4, 9}: reject-heavy, so the allowed side is kept
    words = np.array([(1 << 1) | (1 << 4) | (1 << 9)], np.uint32)
    kind, ids = oracle.adaptive_token_set(words, 10)
    assert kind == oracle.ALLOWS and ids.tolist() == [1, 4, 9]
    # allowed = everything but {0, 7}: accept-heavy, so the refused side is kept
    words = np.array([0x3FF & ~((1 << 0) | (1 << 7))], np.uint32)
    kind, ids = oracle.adaptive_token_set(words, 10)
    assert kind == oracle.DENIES and ids.tolist() == [0, 7]
    # exactly half: the allowed side; bits at and beyond V are never listed
    words = np.array([0b0101010101 | (1 << 20)], np.uint32)
    kind, ids = oracle.adaptive_token_set(words, 10)
    assert kind == oracle.ALLOWS and ids.tolist() == [0, 2, 4, 6, 8]
    # nothing allowed / everything allowed, across a word boundary
    kind, ids = oracle.adaptive_token_set(np.zeros(2, np.uint32), 40)
    assert kind == oracle.ALLOWS and ids.size == 0
    kind, ids = oracle.adaptive_token_set(np.array([0xFFFFFFFF, 0xFF], np.uint32), 40)
    assert kind == oracle.DENIES and ids.size == 0
    kind, ids = oracle.adaptive_token_set(np.array([0xFFFFFFFF, 0x7F], np.uint32), 40)
    assert kind == oracle.DENIES and ids.tolist() == [39]


def test_apply_from_a_token_set_hand_example_and_against_the_dense_apply():
    x = np.arange(1, 7, dtype=np.float32).view(np.uint32).copy()
    y = x.copy()
    oracle.apply_token_set(y, oracle.ALLOWS, np.array([0, 3], np.int32), 6)
    assert y.view(np.float32).tolist() == [1.0, -np.inf, -np.inf, 4.0, -np.inf, -np.inf]
    y = x.copy()
    oracle.apply_token_set(y, oracle.DENIES, np.array([0, 3], np.int32), 6)
    assert y.view(np.float32).tolist() == [-np.inf, 2.0, 3.0, -np.inf, 5.0, 6.0]
    # both storage forms describe the same mask: the result equals the dense apply
    rng = np.random.default_rng(11)
    V = 1003
    for dtype, density in (("bf16", 0.02), ("fp32", 0.97), ("bf16", 0.5)):
        keep = rng.random(V) < density
        words = np.zeros((1, (V + 31) // 32), np.uint32)
        for t in np.nonzero(keep)[0]:
            words[0, t >> 5] |= np.uint32(1 << (t & 31))
        kind, ids = oracle.adaptive_token_set(words[0], V)
        assert kind == (oracle.ALLOWS if 2 * keep.sum() <= V else oracle.DENIES)
        assert ids.size == min(keep.sum(), V - keep.sum())
        logits = make_logits(1, V, dtype, 3)
        raw = logits.view(np.uint32) if dtype == "fp32" else logits
        a, b = raw.copy(), raw.copy()
        oracle.apply_mask(a, words, V)
        oracle.apply_token_set(b[0], kind, ids, V)
        assert (a == b).all()


def test_enum_trie_accepts_exactly_its_strings():
    names = [b'alpha"', b'alps"', b'beta"', b'be"', b'gamma-1"', b'gamma-2"', b'g"']
    op = Sequence(Write(b'"'), enum_trie(names), Write(b";"))
    tree = tree_of(op)
    for n in names:
        assert tree.accepts(list(b'"' + n + b";") + [EOS])
    for bad in [b'alp"', b'alphas"', b'bet"', b'gamma-3"', b'"']:
        assert not tree.accepts(list(b'"' + bad + b";") + [EOS])


# ---------------------------------------------------------------------------------------
# Wait on a multi-byte string (the paper's waits are tokens such as a closing tag)
# ---------------------------------------------------------------------------------------
def test_wait_until_ends_at_the_first_occurrence_of_its_string():
    tree = tree_of(Sequence(Write(b"<p>"), WaitUntil(ALL_BYTES, b"</p>"), Write(b"!")))
    for s, want in [(b"<p>hello</p>!", True), (b"<p></p>!", True), (b"<p>a<b</</p>!", True),
                    (b"<p></p></p>!", False), (b"<p>a</p!", False), (b"<p>a</p>", False)]:
        assert tree.accepts(list(s) + [EOS]) is want, s
    # a string that overlaps itself: the match must restart from the longest border
    tree = tree_of(WaitUntil(SymSet(b"ab"), b"aab"))
    for s, want in [(b"aab", True), (b"aaab", True), (b"abaab", True), (b"bbaaaab", True),
                    (b"aabaab", False), (b"abab", False), (b"acab", False), (b"aa", False)]:
        assert tree.accepts(list(s) + [EOS]) is want, s
    # bytes of the string are accepted even when allow does not list them; deny still rules
    tree = tree_of(WaitUntil(SymSet(b"xy"), b"end", deny=SymSet(b"y")))
    assert tree.accepts(list(b"xxenend") + [EOS]) and not tree.accepts(list(b"xyend") + [EOS])
    for bad in (WaitUntil(ALL_BYTES, b""), WaitUntil(ALL_BYTES, b"ab", deny=SymSet(b"b"))):
        with pytest.raises(oracle.OracleError) as e:
            tree_of(bad)
        assert e.value.code == oracle.ERR_GRAMMAR


def test_wait_until_language_by_plain_string_search():
    # membership by the definition itself: the string occurs, and first occurs at the very end
    until = b"abab"
    tree = tree_of(WaitUntil(SymSet(b"abc"), until))
    for n in range(0, 9):
        for tup in itertools.product(b"abcx", repeat=n):
            s = bytes(tup)
            want = s.endswith(until) and s.find(until) == len(s) - len(until) and b"x" not in s
            assert tree.accepts(list(s) + [EOS]) is want, s


def test_wait_until_mask_closed_form(vocab32k):
    closing = b"</h1>\n"
    op = Sequence(Write(b"<h1>"), WaitUntil(ALL_BYTES, closing), Write(b"<p>"))
    tree = tree_of(op)
    seen = b"so far: 1 <"                       # the text already ends with one byte of the tag
    cursor = tree.walk(tree.start(), list(b"<h1>" + seen))
    got = unpack(oracle.mask(tree, vocab32k, cursor), vocab32k.size)
    n_cut = 0
    for t, tok in enumerate(vocab32k.tokens()):
        if t == 2 or not tok:
            want = False
        else:
            text = seen + tok
            at = text.find(closing)
            if at < 0:
                want = True                      # still inside the slot
            else:                                # what follows the tag must start the next literal
                want = b"<p>".startswith(text[at + len(closing):])
                n_cut += 1
        assert bool(got[t]) == want, tok
    assert got.mean() > 0.95


# ---------------------------------------------------------------------------------------
# token-level Write (the paper's own Write: a token sequence fixed in advance)
# ---------------------------------------------------------------------------------------
def test_token_level_write_allows_exactly_the_next_token_at_token_boundaries():
    tokens = [b"a", b"b", b"", b"ab", b"abX", b"X", b"c", b"cd", b"d", b"Xc", b"bX"]
    vocab = vocab_from_tokens(tokens, eos_id=2)
    X, EOS_ID, B = tokens.index(b"X"), 2, tokens.index(b"b")
    tree = tree_of(Sequence(Write(b"ab"), WriteTokens([X, EOS_ID, B]), Write(b"cd")))

    def allowed(cursor):
        return [tokens[t] if t != 2 else b"<eos>" for t in
                np.flatnonzero(unpack(oracle.mask(tree, vocab, cursor), vocab.size))]

    c = tree.start()
    # "abX" spells the literal and the forced token's bytes, but runs INTO the forced part
    assert allowed(c) == [b"a", b"ab"]
    rc, c1 = oracle.advance(tree, vocab, c, tokens.index(b"a"))
    assert rc == 0 and allowed(c1) == [b"b"]                 # "bX" would run into it as well
    rc, c = oracle.advance(tree, vocab, c, tokens.index(b"ab"))
    assert rc == 0 and allowed(c) == [b"X"]                  # not "Xc": whole token X only
    rc, c = oracle.advance(tree, vocab, c, X)
    assert rc == 0 and allowed(c) == [b"<eos>"]              # the EOS id as a forced token
    rc, c = oracle.advance(tree, vocab, c, EOS_ID)
    assert rc == 0 and allowed(c) == [b"b"]
    rc, bad = oracle.advance(tree, vocab, c, tokens.index(b"a"))
    assert rc == oracle.ERR_REJECTED and bad == c
    rc, c = oracle.advance(tree, vocab, c, B)
    assert rc == 0 and allowed(c) == [b"c", b"cd"]           # byte level again
    rc, c = oracle.advance(tree, vocab, c, tokens.index(b"cd"))
    assert rc == 0 and allowed(c) == [b"<eos>"]
    # a symbol can never enter a forced token
    forced_cursor = tree.walk(tree.start(), list(b"ab"))
    assert oracle.is_dead(tree.step(forced_cursor, ord("X")))
    # an id beyond the vocabulary allows nothing
    lone = tree_of(WriteTokens([99]))
    assert not oracle.mask(lone, vocab, lone.start()).any()


def test_golden_fixture_of_the_section_3_2_listing():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "section_3_2_listing_language.txt")
    tree = tree_of(worked_example_tree())
    n = 0
    for line in open(path):
        line = line.rstrip("\n")
        if not line or line.startswith("#"):
            continue
        verdict, text = line.split(" ", 1)
        text = "" if text == "<empty>" else text
        assert tree.accepts([ord(c) for c in text] + [EOS]) is (verdict == "accept"), line
        n += 1
    assert n >= 15


# ---------------------------------------------------------------------------------------
# random operator trees against the regular-expression restatement
# ---------------------------------------------------------------------------------------
def _random_tree(rng, depth):
    alphabet = b"abcd,;"

    def pick_sets(k):
        """k pairwise disjoint non-empty deciding sets and a stay set disjoint from them."""
        syms = list(alphabet)
        rng.shuffle(syms)
        cases = [SymSet([syms.pop()]) for _ in range(k)]
        if syms and rng.random() < 0.4:
            cases[0] = cases[0] | [syms.pop()]
        stay = SymSet([s for s in syms if rng.random() < 0.5])
        return cases, stay

    def node(d):
        kind = rng.integers(0, 7) if d > 0 else rng.integers(0, 3)
        if kind == 0:
            n = int(rng.integers(1, 4))
            return Write(bytes(rng.choice(list(alphabet), size=n).tolist()))
        if kind == 1:
            (w,), stay = pick_sets(1)
            return Wait(allow=stay | w, wait=w, body=node(d - 1) if d > 0 and rng.random() < 0.3 else None)
        if kind == 2:
            return WaitUntil(SymSet(b"ab,"), bytes(rng.choice(list(b"ab"), size=int(rng.integers(1, 4))).tolist()))
        if kind == 3:
            k = int(rng.integers(2, 4))
            cases, stay = pick_sets(k)
            union = stay
            for c in cases:
                union = union | c
            return Switch(allow=union, cases=cases,
                          bodies=[node(d - 1) if rng.random() < 0.7 else None for _ in range(k)])
        if kind == 4:
            (t, f), stay = pick_sets(2)
            return DoWhile(node(d - 1) if rng.random() < 0.85 else None,
                           Cond(allow=stay | t | f, true_waits=t, false_waits=f))
        return Sequence([node(d - 1) for _ in range(int(rng.integers(0, 4)))])

    return Sequence(node(depth), node(depth - 1))


def test_random_trees_agree_with_their_regular_expression():
    rng = np.random.default_rng(2024)
    alphabet = list(b"abcd,;") + [EOS]
    n_members = 0
    for _ in range(60):
        op = _random_tree(rng, 3)
        tree = tree_of(op)
        prog = regex_ref.program(op)
        for _ in range(120):
            # a random walk that mostly follows accepted symbols, so that deep states are reached
            cursor, text = tree.start(), []
            for _ in range(int(rng.integers(1, 25))):
                options = [s for s in alphabet if not oracle.is_dead(tree.step(cursor, s))]
                if options and rng.random() < 0.85:
                    s = options[int(rng.integers(0, len(options)))]
                else:
                    s = alphabet[int(rng.integers(0, len(alphabet)))]
                nxt = tree.step(cursor, s)
                data = regex_ref.to_bytes(text + [s])
                assert oracle.is_dead(nxt) == (not regex_ref.viable(prog, data)), (op, data)
                if oracle.is_dead(nxt):
                    break
                cursor, text = nxt, text + [s]
            member = regex_ref.member(prog, regex_ref.to_bytes(text))
            assert (cursor == oracle.DONE) == member, (op, text)
            n_members += member
    assert n_members > 200


def test_masks_of_many_rows_equal_the_masks_taken_one_by_one():
    """The multi-row call (threads over rows, strided output) against the single-row call, on
    different trees and cursors per row, with an output whose rows are further apart than W."""
    vocab = make_vocab(4096, seed=7)
    ops = [grammars.html_template(), grammars.json_reference_lookup(doc_nodes=30), grammars.dotted_number()]
    trees = [tree_of(op) for op in ops]
    rng = np.random.default_rng(5)
    row_tree, cursors = [], []
    for r in range(11):
        t = trees[r % 3]
        cur = t.start()
        for _ in range(int(rng.integers(0, 6))):          # a few random live steps
            live = [s for s in range(257) if not oracle.is_dead(t.step(cur, s))]
            if not live:
                break
            nxt = t.step(cur, int(rng.choice(live)))
            if nxt == oracle.DONE:
                break
            cur = nxt
        row_tree.append(t)
        cursors.append(cur)
    W = (vocab.size + 31) // 32
    wide = np.full((11, W + 3), 0xABCDEF01, np.uint32)
    got = oracle.masks(row_tree, vocab, cursors, n_threads=4, out=wide[:, :W])
    for r in range(11):
        assert (got[r] == oracle.mask(row_tree[r], vocab, cursors[r])).all(), r
    assert (wide[:, W:] == 0xABCDEF01).all(), "words between the rows were written"
    assert len({bytes(got[r]) for r in range(11)}) > 3
