"""Templates with holes (host side, no GPU): an instantiated template must accept exactly the
language of the tree in which every hole is replaced by its argument's tree, which the CPU
checker interprets directly.  The two are walked side by side over every reachable transition."""

import numpy as np
import pytest

import oracle
from cosim import co_reachable, mentioned_symbols
from wg_workloads import (ALL_BYTES, DIGITS, EOS, Cond, DoWhile, Hole, IfElse, Sequence, Switch,
                          SymSet, Wait, WaitUntil, Write, WriteTokens, enum_trie, flatten, grammars,
                          substitute)


@pytest.fixture(scope="module")
def wg():
    from paper_2507_16768_b200 import build
    build.build()
    import paper_2507_16768_b200 as wg
    return wg


def check_equal_language(wg, template, args, symbols=None):
    whole = flatten(substitute(template, args))
    tree = oracle.Tree(whole)
    T = wg.Template(flatten(template))
    g = T.instantiate([wg.Grammar(flatten(a)) for a in args])
    syms = symbols or (range(257) if whole.n_nodes < 60 else mentioned_symbols(whole))
    cursor_of = co_reachable(tree, g, syms)
    full = wg.Grammar(whole)
    # every state of the spliced table is in use, and there are as many as a fresh lowering makes
    assert sorted(cursor_of) == list(range(1, g.n_states))
    assert g.n_states == full.n_states and g.n_classes == full.n_classes
    assert cursor_of[g.done_state] == oracle.DONE
    assert g.minimized().n_states == full.minimized().n_states
    return T, g


CASES = {
    "one_hole": (Sequence(Write(b"<a>"), Hole(0), Write(b"</a>")), [enum_trie([b"x1;", b"x22;", b"y;"])]),
    "same_argument_twice": (Sequence(Write(b"<"), Hole(0), Write(b">"), Wait(ALL_BYTES, SymSet(b"<")),
                                     Write(b"/"), Hole(0), Write(b">")),
                            [enum_trie([b"h1", b"h2", b"p!"])]),
    "adjacent_holes": (Sequence(Hole(0), Hole(1), Hole(0), Write(b".")),
                       [Write(b"ab"), Wait(DIGITS, SymSet(b";"))]),
    "hole_first_and_last": (Sequence(Hole(0), Write(b"-"), Hole(1)),
                            [Wait(SymSet(b"xy"), SymSet(b"z")), enum_trie([b"end", b"exit"])]),
    "hole_in_loop_and_branch": (
        Sequence(Write(b"["),
                 DoWhile(Sequence(Write(b'"'), Hole(0)),
                         Cond(SymSet(b",]"), SymSet(b","), SymSet(b"]"))),
                 IfElse(Cond(SymSet(b"+-"), SymSet(b"+"), SymSet(b"-")), Hole(1), None),
                 Wait(ALL_BYTES, SymSet(b"!"), body=Hole(1))),
        [enum_trie([b'1/2"', b'1/3"', b'7"']), Write(b"ok")]),
    "empty_argument": (Sequence(Write(b"a"), Hole(0), Hole(1), Write(b"b"), Hole(0)),
                       [Sequence(), Write(b"")]),
    "only_a_hole": (Hole(0), [Sequence(Write(b"q"), Wait(DIGITS, DIGITS))]),
    "wait_until_and_loops_inside_the_argument": (
        Sequence(Write(b"<p>"), Hole(0), Write(b"\n")),
        [Sequence(WaitUntil(ALL_BYTES, b"</p>"),
                  DoWhile(Write(b"x"), Cond(SymSet(b"+."), SymSet(b"+"), SymSet(b"."))))]),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_instantiated_template_equals_the_substituted_tree(wg, name):
    template, args = CASES[name]
    T, g = check_equal_language(wg, template, args)
    assert T.n_args == len(args)


def test_config5_shape_and_one_static_part_for_every_request(wg):
    template, args0 = grammars.dynamic_snippet_parts(4, n_args=3, enum_size=10)
    T, g0 = check_equal_language(wg, template, args0)
    _, args1 = grammars.dynamic_snippet_parts(5, n_args=3, enum_size=10)
    g1 = T.instantiate([wg.Grammar(flatten(a)) for a in args1])      # the same compiled template
    cursor_of = co_reachable(oracle.Tree(flatten(substitute(template, args1))), g1,
                             mentioned_symbols(flatten(substitute(template, args1))))
    assert sorted(cursor_of) == list(range(1, g1.n_states))
    assert g0.content_hash != g1.content_hash
    # equal arguments give the equal table (and so one grammar id and shared cache entries)
    g0b = T.instantiate([wg.Grammar(flatten(a)) for a in args0])
    assert g0b.content_hash == g0.content_hash and g0b.n_states == g0.n_states


def test_token_level_write_in_template_and_argument(wg):
    template = Sequence(WriteTokens([300, 301]), Hole(0), Write(b"z"), WriteTokens([7]))
    args = [Sequence(Write(b"k"), WriteTokens([400]))]
    whole = flatten(substitute(template, args))
    T = wg.Template(flatten(template))
    g = T.instantiate([wg.Grammar(flatten(args[0]))])
    full = wg.Grammar(whole)
    assert g.n_states == full.n_states
    # walk both tables: forced tokens by id, bytes by symbol
    a, b = g.start_state, full.start_state
    for step in (300, 301, b"k", 400, b"z", 7):
        if isinstance(step, bytes):
            a, b = g.walk(a, step), full.walk(b, step)
        else:
            fa, fb = g.forced_token(a), full.forced_token(b)
            assert fa is not None and fb is not None and fa[0] == fb[0] == step
            a, b = fa[1], fb[1]
        assert a != 0 and b != 0
    assert g.step(a, EOS) == g.done_state and full.step(b, EOS) == full.done_state


def test_regex_fragment_as_argument(wg):
    template = Sequence(Write(b'{"id": "'), Hole(0), Write(b"}"))
    by_hand = Sequence(Wait(DIGITS, DIGITS), Wait(DIGITS | b'"', SymSet(b'"')))     # [0-9]+"
    T = wg.Template(flatten(template))
    g = T.instantiate([wg.Grammar.from_regex(r'[0-9]+"', fragment=True)])
    tree = oracle.Tree(flatten(substitute(template, [by_hand])))
    cursor_of = co_reachable(tree, g, range(257))
    assert sorted(cursor_of) == list(range(1, g.n_states))
    with pytest.raises(wg.WgError) as e:
        wg.Grammar.from_regex(r"[0-9]+", fragment=True)
    assert e.value.status == wg.WG_ERR_GRAMMAR


def test_what_is_refused(wg):
    T = wg.Template(flatten(Sequence(Write(b"a"), Hole(0), Hole(2))))
    assert T.n_args == 3 and T.n_holes == 2
    ok = wg.Grammar(flatten(Write(b"x")))
    with pytest.raises(wg.WgError) as e:
        T.instantiate([ok, ok])                                   # too few arguments
    assert e.value.status == wg.WG_ERR_ARG
    ends_output = wg.Grammar(flatten(Sequence(Write(b"x"), Wait(SymSet([EOS]), SymSet([EOS])))))
    with pytest.raises(wg.WgError) as e:
        T.instantiate([ok, ok, ends_output])                      # an argument that mentions EOS
    assert e.value.status == wg.WG_ERR_GRAMMAR
    with pytest.raises(wg.WgError) as e:
        wg.Grammar(flatten(Sequence(Write(b"a"), Hole(0))))       # holes exist in templates only
    assert e.value.status == wg.WG_ERR_GRAMMAR
    with pytest.raises(oracle.OracleError):
        oracle.Tree(flatten(Hole(0)))                             # the checker knows no holes
    # a saved argument can be loaded and spliced
    g = T.instantiate([ok, ok, wg.Grammar.load(ok.save())])
    assert g.walk(g.start_state, b"axx") != 0 and g.walk(g.start_state, b"ax") != 0
    assert g.step(g.walk(g.start_state, b"axx"), EOS) == g.done_state


def test_instantiation_only_lowers_the_arguments_when_the_static_part_dominates(wg):
    # a long fixed outline with a short enum per section: the shape of the paper's
    # outline-generation task, where the tags are known offline and only titles vary.  What a
    # request still has to lower is counted in table rows (states), not timed: a clock-based
    # comparison would depend on what else the machine is doing.
    parts, args = [], []
    rng = np.random.default_rng(3)
    for i in range(300):
        parts += [Write(b'<section class="outline-level-2" data-index="%d"><h2 id="' % i), Hole(i % 4),
                  Write(b'">'), Wait(ALL_BYTES, SymSet(b"<")), Write(b"/h2></section>\n")]
    for a in range(4):
        names = sorted({bytes(rng.integers(97, 123, size=int(rng.integers(3, 9))).astype(np.uint8)) + b'"'
                        for _ in range(12)})
        args.append(enum_trie(names))
    template = Sequence(parts)
    whole = wg.Grammar(flatten(substitute(template, args)))
    T = wg.Template(flatten(template))
    compiled_args = [wg.Grammar(flatten(a)) for a in args]
    g = T.instantiate(compiled_args)
    assert g.n_states == whole.n_states > 20000
    # per request: four small argument grammars instead of the whole tree
    lowered_per_request = sum(a.n_states for a in compiled_args)
    assert lowered_per_request * 50 < whole.n_states
    assert T.n_states * 2 > whole.n_states - 300 * max(a.n_states for a in compiled_args)
    for probe, alive in ((b'<section class="outline-level-2" data-index="0"><h2 id="', True),
                         (b"<sec", True), (b"<section id", False)):
        assert (g.walk(g.start_state, probe) != 0) == alive == (whole.walk(whole.start_state, probe) != 0)


def _random_op(rng, depth, hole_args=0):
    """A random operator tree over a small alphabet; with hole_args > 0 some leaves are holes."""
    alphabet = b"abcd,;"

    def pick_sets(k):
        syms = list(alphabet)
        rng.shuffle(syms)
        cases = [SymSet([syms.pop()]) for _ in range(k)]
        stay = SymSet([s for s in syms if rng.random() < 0.5])
        return cases, stay

    def node(d):
        if hole_args and rng.random() < 0.25:
            return Hole(int(rng.integers(0, hole_args)))
        kind = rng.integers(0, 6) if d > 0 else rng.integers(0, 2)
        if kind == 0:
            return Write(bytes(rng.choice(list(alphabet), size=int(rng.integers(1, 4))).tolist()))
        if kind == 1:
            (w,), stay = pick_sets(1)
            return Wait(allow=stay | w, wait=w, body=node(d - 1) if d > 0 and rng.random() < 0.3 else None)
        if kind == 2:
            k = int(rng.integers(2, 4))
            cases, stay = pick_sets(k)
            union = stay
            for c in cases:
                union = union | c
            return Switch(allow=union, cases=cases,
                          bodies=[node(d - 1) if rng.random() < 0.7 else None for _ in range(k)])
        if kind == 3:
            (t, f), stay = pick_sets(2)
            return DoWhile(node(d - 1) if rng.random() < 0.85 else None,
                           Cond(allow=stay | t | f, true_waits=t, false_waits=f))
        if kind == 4:
            return WaitUntil(SymSet(b"ab,"), bytes(rng.choice(list(b"ab"), size=int(rng.integers(1, 4))).tolist()))
        return Sequence([node(d - 1) for _ in range(int(rng.integers(0, 4)))])

    return Sequence(node(depth), node(depth - 1))


def test_random_templates_and_arguments(wg):
    rng = np.random.default_rng(77)
    symbols = list(b"abcd,;x") + [EOS]
    checked = holes = 0
    for _ in range(80):
        n_args = int(rng.integers(1, 4))
        template = _random_op(rng, 3, hole_args=n_args)
        args = [_random_op(rng, 2) for _ in range(n_args)]
        whole = flatten(substitute(template, args))
        tree = oracle.Tree(whole)
        T = wg.Template(flatten(template))
        assert T.n_args <= n_args                   # 1 + the largest argument index that occurs
        g = T.instantiate([wg.Grammar(flatten(a)) for a in args[:T.n_args]])
        cursor_of = co_reachable(tree, g, symbols)
        # every reachable cursor has one state; the spliced table has no fewer states than a
        # fresh lowering reaches (copies of an argument that no path enters may be left over)
        full = wg.Grammar(whole)
        assert len(cursor_of) == full.n_states - 1 <= g.n_states - 1
        assert g.minimized().n_states == full.minimized().n_states
        checked += 1
        holes += T.n_holes
    assert checked == 80 and holes > 60
