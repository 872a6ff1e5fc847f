"""GPU parity of the vocabulary-sharded decode step.

Several GPUs that each hold logits[:, v_begin:v_end) are stood in for by several contexts on one
GPU, run one after the other (no kernel waits on another): every "rank" runs
wg_decode_step_shard on its slice, the packed maxima are combined with an element-wise maximum
(what the MAX all-reduce does), and every rank advances with wg_advance_keys.  Masks, masked
logits, tokens and states must equal the CPU checker's on the whole vocabulary, bit for bit."""
import numpy as np
import pytest

import oracle
from cosim import token_symbols
from test_gpu_parity import dev_logits, odd_vocab, raw_bits, to_dev, torch, wg  # noqa: F401
from wg_workloads import flatten, grammars, has_structural_byte, make_logits, make_vocab

pytestmark = pytest.mark.gpu


def run_sharded(wg, torch, vocab, ops, rows, dtype, slices, steps, cache_mode=0, use_cache=True,
                steer=6.0, seed=0):
    from paper_2507_16768_b200.sharding import reduce_best_keys
    V, B = vocab.size, len(rows)
    flats = [flatten(op) for op in ops]
    trees = [oracle.Tree(f) for f in flats]
    grams = [wg.Grammar(f) for f in flats]
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    W = dv.W
    ranks = []
    for (b, e) in slices:
        ctx = wg.Context(dv, 4096 if use_cache else 0, B, cache_mode)
        gids = [ctx.add_grammar(g) for g in grams]
        ranks.append(dict(
            ctx=ctx, b=b, e=e,
            gid=to_dev(torch, np.array([gids[g] for g in rows], np.int32)),
            sid=to_dev(torch, np.array([grams[g].start_state for g in rows], np.int32)),
            mask=torch.zeros((B, W), dtype=torch.int32, device="cuda"),
            keys=torch.zeros(B, dtype=torch.int64, device="cuda"),
            tok=torch.zeros(B, dtype=torch.int32, device="cuda"),
            status=torch.zeros(B, dtype=torch.int32, device="cuda")))
    cursors = [trees[g].start() for g in rows]
    bonus = has_structural_byte(vocab)
    flags = wg.WG_USE_CACHE if use_cache else wg.WG_NO_CACHE
    visited = set()
    for step in range(steps):
        host = make_logits(B, V, dtype, [seed, B], step, bonus, steer)
        want_mask = oracle.masks([trees[g] for g in rows], vocab, cursors, n_threads=8)
        want_tok = oracle.argmax(host, want_mask, V)
        want_logits = host.copy()
        oracle.apply_mask(want_logits, want_mask, V)
        raw_want = want_logits.view(np.uint32) if dtype == "fp32" else want_logits
        shard_logits = []
        for rk in ranks:
            b, e = rk["b"], rk["e"]
            if e <= b:
                rk["keys"].fill_(-(1 << 63))          # a rank without tokens offers nothing
                shard_logits.append(None)
                continue
            dl = dev_logits(torch, np.ascontiguousarray(host[:, b:e]), dtype)
            wg.wg_decode_step_shard(rk["ctx"], rk["gid"], rk["sid"], dl, rk["mask"], b, e,
                                    rk["keys"], flags)
            shard_logits.append(dl)
        best = ranks[0]["keys"].clone()
        for rk in ranks[1:]:
            best = torch.maximum(best, rk["keys"])
        reduce_best_keys(best)                          # one process here: leaves it as it is
        for rk, dl in zip(ranks, shard_logits):
            wg.wg_advance_keys(rk["ctx"], rk["gid"], rk["sid"], best, rk["tok"], rk["status"],
                               wg.WG_RESTART_ON_DONE)
            assert (rk["tok"].cpu().numpy() == want_tok).all(), step
            assert (rk["status"].cpu().numpy() == 0).all()
            if dl is None:
                continue
            b, e = rk["b"], rk["e"]
            assert (raw_bits(torch, dl) == raw_want[:, b:e]).all(), (step, b, e)
            got = rk["mask"].cpu().numpy().view(np.uint32)
            w0, w1 = b // 32, (e + 31) // 32
            assert (got[:, w0:w1] == want_mask[:, w0:w1]).all(), (step, b, e)
            assert (got[:, :w0] == 0).all() and (got[:, w1:] == 0).all()   # other slices untouched
        for r in range(B):
            t = int(want_tok[r])
            rc, cur = oracle.advance(trees[rows[r]], vocab, cursors[r], t)
            assert rc == 0
            cursors[r] = trees[rows[r]].start() if cur == oracle.DONE else cur
            visited.add((rows[r], cursors[r]))
        sids = [rk["sid"].cpu().numpy() for rk in ranks]
        assert all((s == sids[0]).all() for s in sids[1:])
    return ranks, visited


@pytest.mark.parametrize("dtype,cache_mode,use_cache", [("bf16", 0, True), ("fp32", 1, True),
                                                        ("bf16", 0, False)])
def test_three_vocabulary_slices_equal_the_whole(wg, torch, dtype, cache_mode, use_cache):
    from paper_2507_16768_b200.sharding import vocab_slices
    vocab = make_vocab(40000 + 19, seed=23)             # a ragged last slice, V % 32 != 0
    slices = vocab_slices(vocab.size, 3)
    assert slices[0][0] == 0 and slices[-1][1] == vocab.size
    ops = [grammars.html_template(), grammars.json_reference_lookup(doc_nodes=80)]
    rows = [0, 1, 1, 0, 1]
    ranks, visited = run_sharded(wg, torch, vocab, ops, rows, dtype, slices, steps=40,
                                 cache_mode=cache_mode, use_cache=use_cache)
    assert len(visited) > 30
    if use_cache:
        assert all(rk["ctx"].stats()["cache_hits"] > 0 for rk in ranks)


def test_more_ranks_than_slices_and_what_is_refused(wg, torch):
    from paper_2507_16768_b200.sharding import vocab_slices
    vocab = make_vocab(8192 + 100, seed=3)
    slices = vocab_slices(vocab.size, 4)                 # two aligned pieces for four ranks
    assert [e - b for b, e in slices].count(0) == 2
    ranks, _ = run_sharded(wg, torch, vocab, [grammars.html_template()], [0, 0], "fp32", slices,
                           steps=12, steer=8.0)
    rk = next(r for r in ranks if r["e"] - r["b"] > 0 and r["b"] > 0)
    B = 2
    x = torch.zeros((B, vocab.size), dtype=torch.float32, device="cuda")
    for b, e in ((0, 8192), (100, vocab.size), (8192, 9000)):
        with pytest.raises(wg.WgError) as err:      # another slice / unaligned begin / unaligned end
            wg.wg_decode_step_shard(rk["ctx"], rk["gid"], rk["sid"], x[:, :max(1, e - b)], rk["mask"],
                                    b, e, rk["keys"])
        assert err.value.status == wg.WG_ERR_ARG
    with pytest.raises(ValueError):                  # fewer logits columns than the slice has tokens
        wg.wg_decode_step_shard(rk["ctx"], rk["gid"], rk["sid"], x[:, :50], rk["mask"], rk["b"],
                                rk["e"], rk["keys"])
    full = torch.zeros((B, vocab.size), dtype=torch.float32, device="cuda")
    with pytest.raises(wg.WgError):                  # the cache holds one slice's words only
        wg.wg_decode_step(rk["ctx"], rk["gid"], rk["sid"], full, rk["mask"], rk["tok"])
    rk["ctx"].cache_clear()
    wg.wg_decode_step(rk["ctx"], rk["gid"], rk["sid"], full, rk["mask"], rk["tok"])
