"""GPU parity around wg_ctx_remove_grammar (paper Section 3.1: a state machine is instantiated per
request, so a serving process adds and drops grammars for as long as it runs).

Dropping a grammar must leave the other grammars' masks, cached or not, exactly the checker's; the
id must come back for a grammar added later WITHOUT any mask of the old grammar being served for
it; rows that still name the id get an all-zero mask and a status; and many rounds of adding and
dropping must neither exhaust the cache nor slow it into the ground (the hash table is rebuilt
once removed entries hold a quarter of it)."""
import numpy as np
import pytest

import oracle
from test_gpu_parity import dev_logits, raw_bits, to_dev, torch, wg  # noqa: F401
from wg_workloads import flatten, grammars, has_structural_byte, make_logits, make_vocab

pytestmark = pytest.mark.gpu


class Rows:
    """A batch whose rows can change grammar between steps; both sides run side by side."""

    def __init__(self, wg, torch, vocab, ctx, B, dtype="fp32", seed=0):
        self.wg, self.torch, self.vocab, self.ctx, self.B, self.dtype = wg, torch, vocab, ctx, B, dtype
        self.W = (vocab.size + 31) // 32
        self.tree = [None] * B
        self.cursor = [None] * B
        self.gid = np.zeros(B, np.int32)
        self.sid = np.zeros(B, np.int32)
        self.d_mask = torch.zeros((B, self.W), dtype=torch.int32, device="cuda")
        self.d_tok = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.d_status = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.bonus = has_structural_byte(vocab)
        self.seed, self.step_no = seed, 0

    def assign(self, r, tree, gram, gid):
        self.tree[r], self.cursor[r] = tree, tree.start()
        self.gid[r], self.sid[r] = gid, gram.start_state
        self.start = getattr(self, "start", {})
        self.start[r] = (tree.start(), gram.start_state)

    def step(self, dead_rows=()):
        wg, torch, vocab, B = self.wg, self.torch, self.vocab, self.B
        host = make_logits(B, vocab.size, self.dtype, [self.seed, B], self.step_no, self.bonus, 5.0)
        live = [r for r in range(B) if r not in dead_rows]
        want_mask = np.zeros((B, self.W), np.uint32)
        want_mask[live] = oracle.masks([self.tree[r] for r in live], vocab,
                                       [self.cursor[r] for r in live], n_threads=oracle.max_threads())
        want_tok = oracle.argmax(host, want_mask, vocab.size)
        want_logits = host.copy()
        oracle.apply_mask(want_logits, want_mask, vocab.size)
        d_gid, d_sid = to_dev(torch, self.gid), to_dev(torch, self.sid)
        dl = dev_logits(torch, host, self.dtype)
        wg.wg_decode_step(self.ctx, d_gid, d_sid, dl, self.d_mask, self.d_tok, self.d_status,
                          wg.WG_USE_CACHE | wg.WG_RESTART_ON_DONE)
        got_mask = self.d_mask.cpu().numpy().view(np.uint32)
        assert (got_mask == want_mask).all(), self.step_no
        raw_want = want_logits.view(np.uint32) if self.dtype == "fp32" else want_logits
        assert (raw_bits(torch, dl) == raw_want).all(), self.step_no
        tok, status = self.d_tok.cpu().numpy(), self.d_status.cpu().numpy()
        assert (tok == want_tok).all(), self.step_no
        new_sid = d_sid.cpu().numpy()
        for r in range(B):
            if r in dead_rows:
                assert tok[r] == -1 and status[r] != 0 and new_sid[r] == self.sid[r]
                continue
            assert status[r] == 0
            rc, cur = oracle.advance(self.tree[r], vocab, self.cursor[r], int(tok[r]))
            assert rc == 0
            self.cursor[r] = self.start[r][0] if cur == oracle.DONE else cur
        self.sid = new_sid.copy()
        self.step_no += 1


def snippet(seed):
    """A small per-request grammar: the snippet template with three enums of eight names."""
    flat = flatten(grammars.dynamic_snippet_template(seed, n_args=3, enum_size=8))
    return flat, oracle.Tree(flat)


@pytest.mark.parametrize("B,cache_mode", [(6, 0), (80, 0), (80, 1)])
def test_removed_grammar_leaves_the_others_alone_and_its_id_serves_no_stale_mask(wg, torch, B, cache_mode):
    vocab = make_vocab(9000 + 5, seed=31)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, 512, B, cache_mode)
    flat_a, tree_a = snippet(1)
    flat_b, tree_b = snippet(2)
    ga, gb = wg.Grammar(flat_a), wg.Grammar(flat_b)
    ida, idb = ctx.add_grammar(ga), ctx.add_grammar(gb)
    rows = Rows(wg, torch, vocab, ctx, B, "fp32" if cache_mode == 0 else "bf16", seed=B)
    for r in range(B):
        rows.assign(r, *((tree_a, ga, ida) if r % 2 == 0 else (tree_b, gb, idb)))
    for _ in range(25):
        rows.step()
    entries_before = ctx.stats()["cache_entries"]
    ctx.remove_grammar(ida)
    st = ctx.stats()
    assert 0 < st["cache_entries"] < entries_before          # A's masks are gone, B's stay
    with pytest.raises(wg.WgError):
        ctx.remove_grammar(ida)                               # no such grammar any more
    # rows of A now name nothing: zero mask, no token, a status, the state stays; rows of B go on
    ctx.reset_stats()
    rows.step(dead_rows={r for r in range(B) if r % 2 == 0})
    assert ctx.stats()["bad_states"] >= B // 2
    ctx.reset_stats()
    # a new grammar takes A's id; nothing of A may be served for it, from the start state on
    flat_c, tree_c = snippet(3)
    gc = wg.Grammar(flat_c)
    idc = ctx.add_grammar(gc)
    assert idc == ida
    for r in range(0, B, 2):
        rows.assign(r, tree_c, gc, idc)
    for _ in range(25):
        rows.step()
    assert ctx.stats()["rows_uncached"] == 0
    assert ctx.add_grammar(gb) == idb                         # still known by its content


def test_a_long_run_of_requests_that_come_and_go(wg, torch):
    """300 grammars pass through a context that holds few of them at a time: the ids stay small,
    the cache never fills up for good, the hash table is rebuilt on the way, and every step of
    every live row is the checker's."""
    vocab = make_vocab(4000 + 3, seed=37)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    B = 8
    # 256 pool rows, 512 hash slots.  A request lives 24 steps, so the eight live ones hold at most
    # 200 rows; over the run some 6 000 entries are dropped, twelve times the table: without the
    # rebuilds their keys would fill it and every later state would go uncached.
    ctx = wg.Context(dv, 256, B)
    rows = Rows(wg, torch, vocab, ctx, B, "fp32", seed=5)
    live = {}
    for r in range(B):
        flat, tree = snippet(100 + r)
        g = wg.Grammar(flat)
        live[r] = (g, ctx.add_grammar(g))
        rows.assign(r, tree, g, live[r][1])
    max_id = 0
    for round_no in range(300):
        for _ in range(3):
            rows.step()
        r = round_no % B                     # this row's request ends; another one takes its place
        ctx.remove_grammar(live[r][1])
        flat, tree = snippet(1000 + round_no)
        g = wg.Grammar(flat)
        live[r] = (g, ctx.add_grammar(g))
        max_id = max(max_id, live[r][1])
        rows.assign(r, tree, g, live[r][1])
    st = ctx.stats()
    assert max_id < B                        # ids are used again
    assert st["cache_entries"] <= 200 and st["bad_states"] == 0
    assert st["rows_uncached"] == 0 and st["cache_hits"] > 0
