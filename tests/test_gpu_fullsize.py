"""Parity at the full sizes of the workloads, in the launch configuration the benchmark times.

The first and the last step compare EVERY row in full (mask words, masked logits as raw bits,
chosen token); the steps between compare a sample of rows in full and all rows through what
is cheap: the token must be allowed by the checker in the row's cursor, and the device state
must equal the host table walk of that token.
"""
import numpy as np
import pytest

import oracle
from test_gpu_parity import Sim
from wg_workloads import BY_NAME, make_vocab

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


def sample_rows(B, step, n):
    rng = np.random.default_rng(1000 + step)
    rows = {0, B - 1} | set(int(x) for x in rng.choice(B, size=min(n, B), replace=False))
    return sorted(rows)


@pytest.mark.parametrize("cache_mode", [0, 1])        # dense rows, allows / denies entries
def test_json_warm_batch_1024_prewarmed(wg, torch, cache_mode):
    w = BY_NAME["json_warm"]
    vocab = make_vocab(w.V, w.vocab_seed)
    sim = Sim(wg, torch, vocab, [w.grammar(0)], [0] * w.batch, w.dtype,
              cache_capacity=sim_capacity(wg, w), steer=0.0, seed=4, cache_mode=cache_mode)
    sim.ctx.cache_prewarm(sim.gids[0])
    built = sim.ctx.stats()["masks_built"]
    assert built == sim.grams[0].n_states - 1
    sim.ctx.reset_stats()
    for step in range(5):
        sim.step(check_rows=None if step in (0, 4) else sample_rows(w.batch, step, 10))
    st = sim.ctx.stats()
    assert st["masks_built"] == 0, "a prewarmed cache must serve every row"
    assert st["cache_hits"] == 5 * w.batch and st["cache_misses"] == 0
    assert len(sim.visited) > 10


def sim_capacity(wg, w):
    return 4096 if w.use_cache else 0


def test_cold_templates_batch_256_no_cache(wg, torch):
    w = BY_NAME["cold_templates"]
    vocab = make_vocab(w.V, w.vocab_seed)
    ops = [w.grammar(g) for g in range(w.n_grammars)]
    rows = [w.grammar_of_row(r) for r in range(w.batch)]
    sim = Sim(wg, torch, vocab, ops, rows, w.dtype, cache_capacity=0, use_cache=False, seed=3)
    for step in range(4):
        sim.step(check_rows=None if step in (0, 3) else sample_rows(w.batch, step, 14))
    assert sim.ctx.stats()["masks_built"] == 4 * w.batch
    assert len({g for g, _ in sim.visited}) == w.n_grammars


@pytest.mark.parametrize("cache_mode", [0, 1])
def test_dynamic_snippets_batch_128_pairs_share_an_instantiation(wg, torch, cache_mode):
    w = BY_NAME["dynamic_snippets"]
    vocab = make_vocab(w.V, w.vocab_seed)
    n_inst = w.batch // 2
    ops = [w.grammar(g) for g in range(n_inst)]
    rows = [w.grammar_of_row(r) for r in range(w.batch)]
    delays = [w.row_delay(r) for r in range(w.batch)]
    sim = Sim(wg, torch, vocab, ops, rows, w.dtype, cache_capacity=4096, seed=5, steer=6.0,
              delays=delays, cache_mode=cache_mode)
    assert max(g.n_states for g in sim.grams) > 15000
    for step in range(6):
        sim.step(check_rows=None if step in (0, 5) else sample_rows(w.batch, step, 8))
    st = sim.ctx.stats()
    # from the second step on a follower finds what its leader built one step before
    assert st["cache_hits"] >= 5 * n_inst - n_inst
    assert st["rows_uncached"] == 0
