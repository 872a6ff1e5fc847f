"""Parity over whole runs at the full sizes of the workloads, in the launch configuration the
benchmark times (one wg_decode_step per step over the whole batch).

Compared steps check EVERY row in full: mask words, masked logits as raw bits, chosen token,
next state.  The small workloads compare every step.  The large ones compare steps 0-7, every
32nd step (every 64th of the 1 024 steps at batch 1 024) and the last step of the workload's own
step count; the steps between run on logits
drawn on the device and check every row through what is cheap (the token must be accepted by the
checker in the row's cursor, and the device state must equal the host table walk of that token).
Each test asserts that it reached what it is for, e.g. rows in free-text states that allow most
of a vocabulary of 128 256 tokens or more.
"""
import numpy as np
import pytest

import oracle
from cosim import random_walk_states, symbol_representatives
from test_gpu_parity import Sim
from wg_workloads import BY_NAME, flatten, grammars, make_vocab

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def wg():
    import paper_2507_16768_b200 as wg
    return wg


@pytest.fixture(scope="module")
def torch():
    import torch
    torch.cuda.set_device(0)
    return torch


def compared_steps(n_steps, every=32, head=8):
    return set(range(min(head, n_steps))) | set(range(0, n_steps, every)) | {n_steps - 1}


def run(sim, n_steps, compared):
    """Runs the workload's steps; returns the largest allowed fraction seen on a compared row."""
    V = sim.vocab.size
    widest = 0.0
    for step in range(n_steps):
        if step in compared:
            sim.step()
            bits = np.unpackbits(sim.d_mask.cpu().numpy().view(np.uint8), axis=1).sum(axis=1)
            widest = max(widest, float(bits.max()) / V)
        else:
            sim.step_unchecked()
    return widest


def test_html_tiny_every_step(wg, torch):
    w = BY_NAME["html_tiny"]
    vocab = make_vocab(w.V, w.vocab_seed)
    sim = Sim(wg, torch, vocab, [w.grammar(0)], [0], w.dtype, cache_capacity=256, steer=8.0, seed=1)
    widest = run(sim, w.steps, set(range(w.steps)))
    assert widest > 0.5 and len(sim.visited) > 60


def test_json_lookup_every_step_on_all_32_rows(wg, torch):
    w = BY_NAME["json_lookup"]
    vocab = make_vocab(w.V, w.vocab_seed)
    sim = Sim(wg, torch, vocab, [w.grammar(0)], [0] * w.batch, w.dtype, cache_capacity=2048,
              steer=0.0, seed=2)
    run(sim, w.steps, set(range(w.steps)))
    st = sim.ctx.stats()
    assert st["cache_hits"] + st["cache_misses"] == w.steps * w.batch
    # (rows that meet a new state in the same step each build it; one of them files it)
    assert st["masks_built"] >= st["cache_entries"] > 100 and len(sim.visited) > 200
    assert st["rows_uncached"] == 0


def test_cold_templates_batch_256_no_cache(wg, torch):
    w = BY_NAME["cold_templates"]
    vocab = make_vocab(w.V, w.vocab_seed)
    ops = [w.grammar(g) for g in range(w.n_grammars)]
    rows = [w.grammar_of_row(r) for r in range(w.batch)]
    sim = Sim(wg, torch, vocab, ops, rows, w.dtype, cache_capacity=0, use_cache=False, seed=3)
    widest = run(sim, w.steps, compared_steps(w.steps))
    assert sim.ctx.stats()["masks_built"] == w.steps * w.batch
    assert len({g for g, _ in sim.visited}) == w.n_grammars
    # rows in free-text slots: most of the 151 936 tokens allowed, built by the word-wise path
    assert widest > 0.5 and len(sim.visited) > 400


@pytest.mark.parametrize("cache_mode,every", [(0, 64), (1, 128)])   # dense rows, allows / denies
def test_json_warm_batch_1024_prewarmed(wg, torch, cache_mode, every):
    w = BY_NAME["json_warm"]
    vocab = make_vocab(w.V, w.vocab_seed)
    sim = Sim(wg, torch, vocab, [w.grammar(0)], [0] * w.batch, w.dtype, cache_capacity=4096,
              steer=0.0, seed=4, cache_mode=cache_mode)
    sim.ctx.cache_prewarm(sim.gids[0])
    assert sim.ctx.stats()["masks_built"] == sim.grams[0].n_states - 1
    sim.ctx.reset_stats()
    run(sim, w.steps, compared_steps(w.steps, every, head=8 if cache_mode == 0 else 4))
    st = sim.ctx.stats()
    assert st["masks_built"] == 0, "a prewarmed cache must serve every row"
    assert st["cache_hits"] == w.steps * w.batch and st["cache_misses"] == 0
    assert len(sim.visited) > 300


@pytest.mark.parametrize("cache_mode,every", [(0, 32), (1, 128)])
def test_dynamic_snippets_batch_128_pairs_share_an_instantiation(wg, torch, cache_mode, every):
    w = BY_NAME["dynamic_snippets"]
    vocab = make_vocab(w.V, w.vocab_seed)
    n_inst = w.batch // 2
    ops = [w.grammar(g) for g in range(n_inst)]
    rows = [w.grammar_of_row(r) for r in range(w.batch)]
    delays = [w.row_delay(r) for r in range(w.batch)]
    sim = Sim(wg, torch, vocab, ops, rows, w.dtype, cache_capacity=1 << 15, seed=5, steer=6.0,
              delays=delays, cache_mode=cache_mode)
    assert max(g.n_states for g in sim.grams) > 15000
    widest = run(sim, w.steps, compared_steps(w.steps, every, head=8 if cache_mode == 0 else 4))
    st = sim.ctx.stats()
    # from the second step on a follower finds what its leader built one step before
    assert st["cache_hits"] >= (w.steps - 1) * n_inst - n_inst
    assert st["rows_uncached"] == 0
    assert widest > 0.5 and len(sim.visited) > 2000


@pytest.mark.parametrize("cache_mode", [0, 1])
def test_trajectory_on_a_grammar_with_more_than_65535_states(wg, torch, cache_mode):
    """32-bit table entries on the whole step (build, advance).  The rows start in states met on
    random walks, most of them numbered beyond 65 535, and run 64 steps from there."""
    w = BY_NAME["dynamic_snippets"]
    vocab = make_vocab(w.V, w.vocab_seed)
    flat = flatten(grammars.dynamic_snippet_template(0, n_args=16, enum_size=1000))
    tree, g = oracle.Tree(flat), wg.Grammar(flat)
    assert g.n_states > 65535
    rng = np.random.default_rng(29)
    cursor_of = random_walk_states(tree, g, symbol_representatives(flat), rng, n_walks=6,
                                   max_steps=4000)
    high = [s for s in sorted(cursor_of) if s > 65535]
    low = [s for s in sorted(cursor_of) if s <= 65535]
    picks = [high[int(i)] for i in rng.choice(len(high), 12, replace=False)] + \
            [low[int(i)] for i in rng.choice(len(low), 4, replace=False)]
    sim = Sim(wg, torch, vocab, [flat], [0] * len(picks), "fp32", cache_capacity=4096, seed=6,
              steer=6.0, cache_mode=cache_mode, grams=[g],
              starts=[(s, cursor_of[s]) for s in picks])
    for _ in range(64):
        sim.step()
    assert sum(1 for _, s in sim.visited if s > 65535) > 100
    st = sim.ctx.stats()
    assert st["rows_uncached"] == 0 and st["bad_states"] == 0
