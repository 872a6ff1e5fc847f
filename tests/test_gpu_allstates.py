"""Masks of EVERY reachable state of the five workloads' grammars, at the workloads' own
vocabulary sizes, against the CPU checker word for word.

A mask is a function of the operator state alone (paper Section 3.3), so every state can be
checked in isolation: no trajectory has to reach it.  The states go through wg_build_masks in
batches of 1024 rows in shuffled order -- more than 32 rows, so the launch takes 8192-token work
items and every mask spans many of them -- with the cache off, with the dense cache (a pass of
misses, then a pass of hits) and with the compact cache.  Tolerance: none.
"""
import functools

import numpy as np
import pytest

import oracle
from cosim import co_reachable, random_walk_states, symbol_representatives
from wg_workloads import BY_NAME, flatten, grammars, make_vocab

pytestmark = pytest.mark.gpu

BATCH = 1024


@pytest.fixture(scope="module")
def wg():
    import paper_2507_16768_b200 as wg
    return wg


@pytest.fixture(scope="module")
def torch():
    import torch
    torch.cuda.set_device(0)
    return torch


# grammars of a workload that are enumerated (the snippet workload: one of its 64 instantiations)
N_GRAMMARS = {"html_tiny": 1, "json_lookup": 1, "cold_templates": 8, "json_warm": 1,
              "dynamic_snippets": 1}
# workloads with free-text slots must show a state that allows most of the vocabulary
HAS_FREE_TEXT = {"html_tiny", "cold_templates", "dynamic_snippets"}


@functools.lru_cache(maxsize=1)
def checker_side(name):
    """(vocab, flats, [(grammar index, library state, cursor)], expected masks [N, W])."""
    import paper_2507_16768_b200 as wg
    w = BY_NAME[name]
    vocab = make_vocab(w.V, w.vocab_seed)
    flats, trees, rows = [], [], []
    for gi in range(N_GRAMMARS[name]):
        flat = flatten(w.grammar(gi))
        tree, g = oracle.Tree(flat), wg.Grammar(flat)
        cursor_of = co_reachable(tree, g, symbol_representatives(flat))
        assert len(cursor_of) == g.n_states - 1, "every live state of the table is reachable"
        flats.append(flat)
        trees.append(tree)
        rows += [(gi, s, cursor_of[s]) for s in sorted(cursor_of)]
    want = oracle.masks([trees[gi] for gi, _, _ in rows], vocab, [c for _, _, c in rows],
                        n_threads=oracle.max_threads())
    return vocab, flats, rows, want


def compare_all(wg, torch, ctx, gids, rows, want, flags, order):
    """wg_build_masks over all rows in the given order, BATCH rows a call; every word compared."""
    W = want.shape[1]
    gid_all = np.array([gids[gi] for gi, _, _ in rows], np.int32)
    sid_all = np.array([s for _, s, _ in rows], np.int32)
    for first in range(0, len(order), BATCH):
        idx = order[first:first + BATCH]
        out = torch.full((len(idx), W), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
        wg.wg_build_masks(ctx, torch.from_numpy(gid_all[idx]).cuda(),
                          torch.from_numpy(sid_all[idx]).cuda(), out, flags)
        expect = torch.from_numpy(want[idx].view(np.int32)).cuda()
        if not torch.equal(out, expect):
            bad = (out != expect).any(dim=1).nonzero().flatten().cpu().tolist()
            raise AssertionError(f"masks differ for rows {[rows[idx[b]][:2] for b in bad[:8]]}")


@pytest.mark.parametrize("name", ["html_tiny", "json_lookup", "cold_templates", "json_warm",
                                  "dynamic_snippets"])
def test_masks_of_every_state_at_the_workloads_own_size(wg, torch, name):
    w = BY_NAME[name]
    vocab, flats, rows, want = checker_side(name)
    V, W = vocab.size, want.shape[1]
    allowed = np.unpackbits(want.view(np.uint8), axis=1).sum(axis=1)
    assert allowed.min() >= 1, "a reachable state allows at least one token"
    if name in HAS_FREE_TEXT:
        assert allowed.max() > V // 2, "a free-text state allows most of the vocabulary"
    if V >= 128256:
        assert W * 32 > 8 * 8192 and len(rows) > 32   # many 8192-token items per mask
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    grams = [wg.Grammar(f) for f in flats]
    rng = np.random.default_rng(17)
    order = rng.permutation(len(rows))
    # cache off
    ctx = wg.Context(dv, 0, BATCH)
    gids = [ctx.add_grammar(g) for g in grams]
    compare_all(wg, torch, ctx, gids, rows, want, wg.WG_NO_CACHE, order)
    assert ctx.stats()["masks_built"] == len(rows)
    del ctx
    # dense and compact cache: a pass that builds every state, then a pass served from the cache
    for mode in (wg.WG_CACHE_DENSE, wg.WG_CACHE_COMPACT):
        ctx = wg.Context(dv, len(rows) + 8, BATCH, mode, 0)
        gids = [ctx.add_grammar(g) for g in grams]
        compare_all(wg, torch, ctx, gids, rows, want, wg.WG_USE_CACHE, order)
        st = ctx.stats()
        assert st["masks_built"] == len(rows) and st["rows_uncached"] == 0, (mode, st)
        compare_all(wg, torch, ctx, gids, rows, want, wg.WG_USE_CACHE, rng.permutation(len(rows)))
        st = ctx.stats()
        assert st["masks_built"] == len(rows) and st["cache_hits"] == len(rows), (mode, st)
        del ctx
    checker_side.cache_clear()


def test_masks_of_a_grammar_with_more_than_65535_states(wg, torch):
    """Tables beyond 65 535 states are stored with 32-bit entries: a different instantiation of
    the walk, the per-state set-up and the advance.  16 sections with enums of 1000 names each
    (the snippet workload taken literally, a quarter of its sections) give about 100 000 states;
    the states met on random walks are compared, those numbered beyond 65 535 among them."""
    w = BY_NAME["dynamic_snippets"]
    vocab = make_vocab(w.V, w.vocab_seed)
    flat = flatten(grammars.dynamic_snippet_template(0, n_args=16, enum_size=1000))
    tree, g = oracle.Tree(flat), wg.Grammar(flat)
    assert g.n_states > 65535
    rng = np.random.default_rng(23)
    cursor_of = random_walk_states(tree, g, symbol_representatives(flat), rng, n_walks=24,
                                   max_steps=4000)
    sids = sorted(cursor_of)
    assert len(sids) > 2000 and sum(s > 65535 for s in sids) > 300
    rows = [(0, s, cursor_of[s]) for s in sids]
    want = oracle.masks([tree] * len(rows), vocab, [c for _, _, c in rows],
                        n_threads=oracle.max_threads())
    allowed = np.unpackbits(want.view(np.uint8), axis=1).sum(axis=1)
    assert allowed.min() >= 1 and allowed.max() > vocab.size // 2
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    order = rng.permutation(len(rows))
    for mode, flags in ((wg.WG_CACHE_DENSE, wg.WG_NO_CACHE), (wg.WG_CACHE_DENSE, wg.WG_USE_CACHE),
                        (wg.WG_CACHE_COMPACT, wg.WG_USE_CACHE)):
        ctx = wg.Context(dv, len(rows) + 8, BATCH, mode, 0)
        gids = [ctx.add_grammar(g)]
        compare_all(wg, torch, ctx, gids, rows, want, flags, order)
        if flags == wg.WG_USE_CACHE:
            compare_all(wg, torch, ctx, gids, rows, want, flags, order[::-1])
            assert ctx.stats()["cache_hits"] == len(rows)
        del ctx
