"""GPU parity of the compact (allows / denies) mask cache against the CPU checker.

Every result of a WG_CACHE_COMPACT context must equal the checker's bit for bit, exactly as
with dense cache rows; in addition each cached entry, read back as a token set, must be the
set the checker derives from its own mask by the paper's rule (Section 3.3).
"""
import numpy as np
import pytest

import oracle
from cosim import co_reachable, mentioned_symbols
from test_gpu_parity import SMALL, Sim, dev_logits, odd_vocab, raw_bits, to_dev, torch, wg  # noqa: F401
from wg_workloads import BY_NAME, flatten, grammars, make_logits, make_vocab

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", sorted(SMALL))
def test_entries_are_the_checkers_token_sets_and_expand_to_its_masks(wg, torch, name):
    vocab = odd_vocab()
    flat = flatten(SMALL[name]())
    tree = oracle.Tree(flat)
    g = wg.Grammar(flat)
    cursor_of = co_reachable(tree, g, mentioned_symbols(flat))
    sids = sorted(cursor_of)
    want = oracle.masks([tree] * len(sids), vocab, [cursor_of[s] for s in sids], n_threads=8)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, cache_capacity=g.n_states, max_batch=64, cache_mode=wg.WG_CACHE_COMPACT)
    gid = ctx.add_grammar(g)
    ctx.cache_prewarm(gid)
    st = ctx.stats()
    assert st["cache_entries"] == g.n_states - 1 and st["rows_uncached"] == 0
    assert 0 < st["cache_bytes"] < (g.n_states - 1) * dv.W * 4 // 2
    kinds = set()
    for i, s in enumerate(sids[:: max(1, len(sids) // 40)]):
        i = sids.index(s)
        kind, ids, nbytes = ctx.cache_entry(gid, s)
        want_kind, want_ids = oracle.adaptive_token_set(want[i], vocab.size)
        assert kind == want_kind and np.array_equal(ids, want_ids), (name, s)
        n_spans = (dv.W + 31) // 32
        assert 8 * n_spans <= nbytes <= 8 * n_spans + 4 * min(ids.size, dv.W)
        kinds.add(kind)
    assert ctx.cache_entry(gid, g.n_states + 7) is None
    if name == "html":                              # literal states and free-text slots
        assert kinds == {wg.WG_ENTRY_ALLOWS, wg.WG_ENTRY_DENIES}
    # the standalone mask call expands entries into rows (all hits after the prewarm)
    for first in range(0, len(sids), 64):
        chunk = sids[first:first + 64]
        out = torch.full((len(chunk), dv.W + 3), -1, dtype=torch.int32, device="cuda")
        wg.wg_build_masks(ctx, torch.full((len(chunk),), gid, dtype=torch.int32, device="cuda"),
                          to_dev(torch, np.array(chunk, np.int32)), out)
        got = out.cpu().numpy().view(np.uint32)
        assert (got[:, :dv.W] == want[first:first + len(chunk)]).all()
        assert (got[:, dv.W:] == 0xFFFFFFFF).all()
    assert ctx.stats()["masks_built"] == g.n_states - 1


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_rows_masked_from_entries_equal_the_checkers_apply_from_token_sets(wg, torch, dtype):
    vocab = make_vocab(8192 + 40, seed=12)          # rows stay 16-byte aligned: the fast kernel
    flat = flatten(grammars.html_template())
    tree = oracle.Tree(flat)
    g = wg.Grammar(flat)
    cursor_of = co_reachable(tree, g, mentioned_symbols(flat))
    sids = sorted(cursor_of)[:48]
    B, V = len(sids), vocab.size
    want_mask = oracle.masks([tree] * B, vocab, [cursor_of[s] for s in sids], n_threads=8)
    host = make_logits(B, V, dtype, [3, B], 0)
    want = (host.view(np.uint32) if dtype == "fp32" else host).copy()
    for r in range(B):
        kind, ids = oracle.adaptive_token_set(want_mask[r], V)
        oracle.apply_token_set(want[r], kind, ids, V)
    want_tok = oracle.argmax(host, want_mask, V)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, cache_capacity=256, max_batch=B, cache_mode=wg.WG_CACHE_COMPACT)
    gid = ctx.add_grammar(g)
    d_gid = torch.full((B,), gid, dtype=torch.int32, device="cuda")
    for attempt in range(2):                         # first all misses, then all hits
        d_sid = to_dev(torch, np.array(sids, np.int32))
        dl = dev_logits(torch, host, dtype)
        mask = torch.zeros((B, dv.W), dtype=torch.int32, device="cuda")
        tok = torch.zeros(B, dtype=torch.int32, device="cuda")
        wg.wg_decode_step(ctx, d_gid, d_sid, dl, mask, tok)
        assert (raw_bits(torch, dl) == want).all(), attempt
        assert (mask.cpu().numpy().view(np.uint32) == want_mask).all()
        assert (tok.cpu().numpy() == want_tok).all()
    st = ctx.stats()
    assert st["cache_hits"] == B and st["cache_misses"] == B and st["masks_built"] == B


@pytest.mark.parametrize("dtype,fused", [("bf16", True), ("fp32", True), ("bf16", False)])
def test_trajectories_with_a_compact_cache(wg, torch, dtype, fused):
    vocab = odd_vocab()                              # V % 32 != 0 and unaligned rows
    ops = [grammars.html_template(), grammars.json_reference_lookup(doc_nodes=60),
           grammars.random_template(1)]
    rows = [0, 1, 2, 1, 0, 2, 2, 1, 1]
    sim = Sim(wg, torch, vocab, ops, rows, dtype, cache_capacity=4096, seed=5,
              cache_mode=wg.WG_CACHE_COMPACT)
    for _ in range(40):
        sim.step(fused=fused)
    st = sim.ctx.stats()
    assert st["cache_hits"] > 0 and st["rows_uncached"] == 0
    assert st["cache_bytes"] < st["cache_entries"] * sim.W * 4


def test_aligned_rows_trajectory_with_a_compact_cache(wg, torch):
    w = BY_NAME["html_tiny"]
    vocab = make_vocab(w.V, w.vocab_seed)
    sim = Sim(wg, torch, vocab, [w.grammar(0)], [0, 0, 0], w.dtype, cache_capacity=256, steer=8.0,
              seed=2, cache_mode=wg.WG_CACHE_COMPACT)
    for i in range(80):
        sim.step(fused=(i % 5 != 0))
    assert len(sim.visited) > 30


def test_a_full_arena_leaves_states_uncached_and_results_unchanged(wg, torch):
    vocab = make_vocab(8192, seed=9)
    ops = [grammars.random_template(s) for s in range(3)]
    rows = [0, 1, 2, 0, 1, 2, 2, 2, 1, 0, 0]
    # the arena never holds less than one mask with every word stored (1 KB here), which is
    # room for a handful of the small entries these states make
    sim = Sim(wg, torch, vocab, ops, rows, "bf16", cache_capacity=4096, seed=3,
              cache_mode=wg.WG_CACHE_COMPACT, arena_bytes=1)
    for _ in range(30):
        sim.step()
    st = sim.ctx.stats()
    assert st["rows_uncached"] > 0 and st["cache_hits"] > 0
    assert st["cache_bytes"] <= 4 * 256 + st["cache_entries"] * 8 * 8   # arena + span headers
    sim.ctx.cache_clear()
    assert sim.ctx.stats()["cache_bytes"] == 0
    for _ in range(5):
        sim.step()


def test_compact_mode_is_refused_on_a_dense_context_read(wg, torch):
    vocab = make_vocab(4096, seed=4)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, cache_capacity=8, max_batch=4)
    with pytest.raises(wg.WgError) as e:
        ctx.cache_entry(0, 1)
    assert e.value.status == wg.WG_ERR_ARG
    with pytest.raises(wg.WgError):
        wg.Context(dv, 8, 4, cache_mode=7)
