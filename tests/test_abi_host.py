"""Host-side checks that need no GPU: the library loads and exports what wg.h declares, and
the operator-to-table lowering agrees with the CPU checker transition by transition."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from cosim import co_reachable, mentioned_symbols
from wg_workloads import (ALL_BYTES, EOS, Cond, DoWhile, IfElse, Sequence, SymSet, Wait, WaitUntil,
                          Write, WriteTokens, flatten, grammars, make_vocab)

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def wg():
    from paper_2507_16768_b200 import build
    build.build()
    import paper_2507_16768_b200 as wg
    return wg


def test_library_exports_every_declared_symbol(wg):
    header = open(os.path.join(ROOT, "include", "wg.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(wg_[a-z0-9_]+)\s*\(", header))
    assert {"wg_load_vocab", "wg_compile_grammar", "wg_build_masks", "wg_mask_cache_lookup",
            "wg_apply_mask", "wg_advance"} <= declared
    lib = ctypes.CDLL(wg.binding.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in wg.h but not exported"
    assert declared == set(wg.binding.EXPORTED)


def test_strerror_and_launch_counter(wg):
    lib = ctypes.CDLL(wg.binding.LIB_PATH)
    lib.wg_strerror.restype = ctypes.c_char_p
    assert lib.wg_strerror(0) == b"ok"
    assert b"grammar" in lib.wg_strerror(-2)
    assert wg.kernel_launch_count() >= 0


GRAMMARS = {
    "dotted_number": grammars.dotted_number,
    "html": grammars.html_template,
    "json_generic": lambda: grammars.json_reference_lookup(doc_nodes=0),
    "json_doc": lambda: grammars.json_reference_lookup(doc_nodes=120),
    "template1": lambda: grammars.random_template(1),
    "template6": lambda: grammars.random_template(6),
    "snippets": lambda: grammars.dynamic_snippet_template(2, n_args=3, enum_size=12),
    "html_tags": lambda: grammars.html_template(wait_for_tag=True),
    "overlapping_until": lambda: Sequence(WaitUntil(SymSet(b"abc"), b"abcab", body=Write(b"x")),
                                          WaitUntil(ALL_BYTES, b"aa")),
    "empty_bodies": lambda: Sequence(
        Write(b""), DoWhile(None, Cond(ALL_BYTES, SymSet(b","), SymSet(b";"))),
        Wait(SymSet(b"ab"), SymSet(b"!"), body=Sequence()), IfElse(
            Cond(SymSet(b"xyz"), SymSet(b"y"), SymSet(b"z")), None, Sequence(Write(b""))),
        Write(b"end")),
}


@pytest.mark.parametrize("name", sorted(GRAMMARS))
def test_lowered_table_matches_checker_on_every_reachable_transition(wg, name):
    op = GRAMMARS[name]()
    flat = flatten(op)
    tree = oracle.Tree(flat)
    g = wg.Grammar(flat)
    symbols = range(257) if flat.n_nodes < 60 else mentioned_symbols(flat)
    cursor_of = co_reachable(tree, g, symbols)
    # every table state is reachable and was paired (state 0 is DEAD)
    assert sorted(cursor_of) == list(range(1, g.n_states))
    assert g.start_state == 1
    assert cursor_of[g.done_state] == oracle.DONE
    assert g.step(g.done_state, EOS) == g.done_state
    assert all(g.step(0, s) == 0 for s in (0, 65, EOS))
    assert g.step(g.n_states, 65) == 0 and g.step(1, 257) == 0 and g.step(-1, 0) == 0


def test_identical_trees_hash_equal_and_different_trees_do_not(wg):
    a = wg.Grammar(flatten(grammars.random_template(3)))
    b = wg.Grammar(flatten(grammars.random_template(3)))
    c = wg.Grammar(flatten(grammars.random_template(4)))
    assert a.content_hash == b.content_hash != c.content_hash


@pytest.mark.parametrize("bad", [
    Wait(allow=SymSet(b"a"), wait=SymSet()),
    Wait(allow=SymSet(b"ab"), wait=SymSet(b"b"), deny=SymSet(b"b")),
    IfElse(Cond(SymSet(b"ab"), SymSet(b"ab"), SymSet(b"b")), None, None),
    DoWhile(Write(b"x"), Cond(SymSet(b"a"), SymSet(b"a"), SymSet())),
    WaitUntil(ALL_BYTES, b""),
    WaitUntil(ALL_BYTES, b"ab", deny=SymSet(b"a")),
])
def test_compile_rejects_what_the_checker_rejects(wg, bad):
    flat = flatten(bad)
    with pytest.raises(oracle.OracleError) as oe:
        oracle.Tree(flat)
    with pytest.raises(wg.WgError) as we:
        wg.Grammar(flat)
    assert oe.value.code == oracle.ERR_GRAMMAR and we.value.status == wg.binding.WG_ERR_GRAMMAR


def test_compile_rejects_malformed_arrays(wg):
    flat = flatten(Sequence(Write(b"a"), Write(b"b")))
    flat.children[1] = flat.children[0]
    with pytest.raises(wg.WgError) as e:
        wg.Grammar(flat)
    assert e.value.status == wg.binding.WG_ERR_GRAMMAR
    flat = flatten(Sequence(Write(b"a"), Write(b"b")))
    flat.nodes[1, 6] = 99          # literal runs past the data array
    with pytest.raises(wg.WgError) as e:
        wg.Grammar(flat)
    assert e.value.status == wg.binding.WG_ERR_ARG
    flat = flatten(Write(b"a"))
    flat.root = 5
    with pytest.raises(wg.WgError):
        wg.Grammar(flat)


def test_large_enum_grammar_needs_wide_state_ids(wg):
    g = wg.Grammar(flatten(grammars.dynamic_snippet_template(0, n_args=8, enum_size=1000)))
    assert g.n_states > 40000


def test_token_level_write_states_follow_the_checker_token_by_token(wg):
    vocab = make_vocab(3000, seed=17)
    toks = vocab.tokens()
    digits = SymSet(b"0123456789")
    op = Sequence(Write(b"id="), WriteTokens([500, 2, 501]),
                  DoWhile(Sequence(WriteTokens([600]), Wait(digits, digits)),
                          Cond(digits | b",.", SymSet(b","), SymSet(b"."))),
                  WriteTokens([]), Write(b"ok"))
    flat = flatten(op)
    tree, g = oracle.Tree(flat), wg.Grammar(flat)
    assert wg.Grammar(flat).content_hash == g.content_hash
    rng = np.random.default_rng(3)
    for _ in range(20):
        cursor, sid = tree.start(), g.start_state
        for _ in range(40):
            words = oracle.mask(tree, vocab, cursor)
            allowed = np.flatnonzero(np.unpackbits(words.view(np.uint8), bitorder="little")[:vocab.size])
            assert allowed.size > 0
            forced = g.forced_token(sid)
            if forced is not None:
                assert allowed.tolist() == [forced[0]]
            # also try a few tokens that are not allowed: both sides must refuse them
            for t in rng.integers(0, vocab.size, size=5):
                rc, _ = oracle.advance(tree, vocab, cursor, int(t))
                syms = [EOS] if t == vocab.eos_id else list(toks[t])
                assert (rc == 0) == (g.step_token(sid, int(t), syms) != 0 and len(syms) > 0)
            t = int(rng.choice(allowed))
            rc, cursor = oracle.advance(tree, vocab, cursor, t)
            sid = g.step_token(sid, t, [EOS] if t == vocab.eos_id else list(toks[t]))
            assert rc == 0 and sid != 0
            if cursor == oracle.DONE:
                assert sid == g.done_state
                break
    bad = flatten(WriteTokens([3]))
    bad.data[:] = np.frombuffer(np.array([-4], "<i4").tobytes(), np.uint8)
    with pytest.raises(wg.WgError) as e:
        wg.Grammar(bad)
    assert e.value.status == wg.binding.WG_ERR_GRAMMAR


def test_header_compiles_as_plain_c(tmp_path):
    import subprocess
    src = tmp_path / "use_wg.c"
    src.write_text('#include "wg.h"\n'
                   'int probe(void) { wg_stats s; wg_op_node n; (void)s; (void)n;\n'
                   '  return WG_OK + WG_DTYPE_BF16 + WG_OP_WRITE_TOKENS + (int)sizeof(wg_op_node); }\n')
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-c",
                           "-I", os.path.join(ROOT, "include"), str(src), "-o",
                           str(tmp_path / "use_wg.o")])


@pytest.mark.parametrize("name", ["dotted_number", "html", "json_doc", "template1", "snippets",
                                  "html_tags", "overlapping_until", "empty_bodies"])
def test_minimized_grammar_keeps_the_language(wg, name):
    flat = flatten(GRAMMARS[name]())
    tree = oracle.Tree(flat)
    g = wg.Grammar(flat)
    m = g.minimized()
    assert m.n_states <= g.n_states and m.start_state == 1
    symbols = range(257) if flat.n_nodes < 60 else mentioned_symbols(flat)
    cursor_of = co_reachable(tree, m, symbols)          # checks every transition against the checker
    assert sorted(cursor_of) == list(range(1, m.n_states))
    assert cursor_of[m.done_state] == oracle.DONE
    again = m.minimized()
    assert again.n_states == m.n_states and again.content_hash == m.content_hash


def test_minimization_merges_repeated_tails(wg):
    g = wg.Grammar(flatten(grammars.json_reference_lookup()))
    assert g.minimized().n_states < g.n_states // 4
    r = wg.Grammar.from_regex(r"(a\d*|b)c(x|y)?z")      # the front end copies tails into branches
    assert r.minimized().n_states < r.n_states
    # forced tokens stay apart by token id
    t = wg.Grammar(flatten(Sequence(WriteTokens([5, 6, 5, 6]), Write(b"ab"))))
    m = t.minimized()
    assert m.n_states == t.n_states
    assert [m.forced_token(s)[0] for s in range(1, 5)] == [5, 6, 5, 6]


def test_saved_grammar_loads_back_identical_and_damage_is_refused(wg):
    for op in (grammars.json_reference_lookup(doc_nodes=50), Sequence(Write(b"a"), WriteTokens([7, 9]))):
        g = wg.Grammar(flatten(op))
        blob = g.save()
        back = wg.Grammar.load(blob)
        assert (back.n_states, back.n_classes, back.start_state, back.done_state, back.content_hash) == \
               (g.n_states, g.n_classes, g.start_state, g.done_state, g.content_hash)
        for s_ in range(g.n_states):
            assert back.forced_token(s_) == g.forced_token(s_)
            for sym in (0, 34, 48, 97, 255, EOS):
                assert back.step(s_, sym) == g.step(s_, sym)
        assert wg.Grammar.load(back.save()).save() == blob
        for damaged in (blob[:-1], blob + b"x", b"\0" * len(blob), blob[:4] + b"\x09" + blob[5:]):
            with pytest.raises(wg.WgError) as e:
                wg.Grammar.load(damaged)
            assert e.value.status == wg.binding.WG_ERR_ARG
        # a table entry pointing outside the table
        bad = bytearray(blob)
        off = 40 + 256 + 4 * g.n_classes            # first cell of state 1
        bad[off:off + 4] = (g.n_states + 5).to_bytes(4, "little")
        with pytest.raises(wg.WgError):
            wg.Grammar.load(bytes(bad))
        # damage that keeps every field in range is caught by the content hash: a stored hash
        # that is not the hash of the contents, and a changed symbol-class map (the header is 48
        # bytes with the hash in its last 8; the class map follows)
        wrong_hash = bytearray(blob)
        wrong_hash[40] ^= 1
        swapped = bytearray(blob)
        swapped[48 + ord("a")], swapped[48 + ord("b")] = swapped[48 + ord("b")], swapped[48 + ord("a")]
        assert bytes(swapped) != blob
        for damaged in (wrong_hash, swapped):
            with pytest.raises(wg.WgError) as e:
                wg.Grammar.load(bytes(damaged))
            assert e.value.status == wg.binding.WG_ERR_ARG


def test_random_trees_lower_to_tables_that_match_the_checker(wg):
    from test_oracle_pins import _random_tree
    rng = np.random.default_rng(77)
    symbols = list(b"abcd,;x") + [EOS]
    for _ in range(80):
        flat = flatten(_random_tree(rng, 3))
        tree, g = oracle.Tree(flat), wg.Grammar(flat)
        cursor_of = co_reachable(tree, g, symbols)
        assert sorted(cursor_of) == list(range(1, g.n_states))
        m = g.minimized()
        assert sorted(co_reachable(tree, m, symbols)) == list(range(1, m.n_states))
