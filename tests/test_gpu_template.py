"""GPU parity for instantiated templates: the decode path runs on tables made by splicing
compiled arguments into a compiled template, the CPU checker interprets the tree in which the
holes are replaced by the arguments' trees.  Masks, masked logits, tokens and states must agree
bit for bit."""
import pytest

from test_gpu_parity import Sim, torch, wg  # noqa: F401
from wg_workloads import flatten, grammars, make_vocab, substitute

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cache_mode", [0, 1])
def test_trajectories_on_instantiated_templates(wg, torch, cache_mode):
    vocab = make_vocab(16384, seed=5)
    template, _ = grammars.dynamic_snippet_parts(0, n_args=4, enum_size=12)
    T = wg.Template(flatten(template))
    requests = [grammars.dynamic_snippet_parts(seed, n_args=4, enum_size=12)[1] for seed in (1, 2, 3)]
    whole = [substitute(template, args) for args in requests]
    grams = [T.instantiate([wg.Grammar(flatten(a)) for a in args]) for args in requests]
    rows = [0, 0, 1, 1, 2, 2, 0, 1]
    sim = Sim(wg, torch, vocab, whole, rows, "fp32", cache_capacity=4096, seed=8, steer=7.0,
              delays=[0, 1, 0, 1, 0, 1, 0, 0], grams=grams, cache_mode=cache_mode)
    for i in range(60):
        sim.step(fused=(i % 4 != 0))
    st = sim.ctx.stats()
    assert st["cache_hits"] > 0 and st["rows_uncached"] == 0
    assert len(sim.visited) > 40
    # a second instantiation with the same arguments is the same grammar to the context
    again = T.instantiate([wg.Grammar(flatten(a)) for a in requests[0]])
    assert sim.ctx.add_grammar(again) == sim.gids[0]
