"""GPU parity: the CUDA library against the CPU checker, bit for bit, through the C ABI.

Tolerance: none.  Masks, masked logits (raw bit patterns), chosen tokens and states must be
identical on the same seeded inputs.
"""
import numpy as np
import pytest

import oracle
from cosim import co_reachable, mentioned_symbols, token_symbols
from wg_workloads import (ALL_BYTES, BY_NAME, EOS, Cond, DoWhile, Sequence, SymSet, Wait, Write,
                          WriteTokens, flatten, grammars,
                          has_structural_byte, make_logits, make_vocab, vocab_from_tokens)

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


def to_dev(torch, a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def dev_logits(torch, host, dtype):
    """Upload logits generated on the host; bf16 arrives as raw uint16 bit patterns."""
    if dtype == "bf16":
        return torch.from_numpy(host.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(host).cuda()


def raw_bits(torch, t):
    """Device logits back to host as raw bit patterns (uint16 / uint32)."""
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.view(torch.int32).cpu().numpy().view(np.uint32)


def odd_vocab():
    """A vocabulary whose size is not a multiple of 32 and that holds tokens beyond 16 bytes."""
    base = make_vocab(5000, seed=21)
    toks = base.tokens()
    extra = [b"<h1 class=\"document-title\" id=\"outline-root\">", b"section-title\" id=\"outline-",
             b"a" * 17, b"x" * 40 + b"<", b"  " * 9 + b"</p>\n<h2 class=", b"0123456789/0123456789",
             b'{"topic": 12, "paths": ["1/2', b"q" * 300, b"", b"</h1>\n<p class=\"document-abs",
             # a slot's closing byte as the last byte of the 16-byte record, and one byte before it
             b"a" * 15 + b"</h1>\n", b"a" * 14 + b"</", b"a" * 15 + b"<", b"b" * 16 + b"</p>"]
    return vocab_from_tokens(toks + extra, eos_id=2)


SMALL = {
    "html": grammars.html_template,
    "json_doc": lambda: grammars.json_reference_lookup(doc_nodes=150),
    "json_generic": lambda: grammars.json_reference_lookup(doc_nodes=0),
    "template2": lambda: grammars.random_template(2),
    "snippets": lambda: grammars.dynamic_snippet_template(4, n_args=3, enum_size=10),
    "dotted_number": grammars.dotted_number,
    "html_tags": lambda: grammars.html_template(wait_for_tag=True),
}


@pytest.mark.parametrize("name", sorted(SMALL))
def test_masks_of_every_state_match(wg, torch, name):
    vocab = odd_vocab()
    assert vocab.size % 32 != 0
    flat = flatten(SMALL[name]())
    tree = oracle.Tree(flat)
    g = wg.Grammar(flat)
    cursor_of = co_reachable(tree, g, mentioned_symbols(flat))
    sids = sorted(cursor_of)
    want = oracle.masks([tree] * len(sids), vocab, [cursor_of[s] for s in sids], n_threads=8)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, cache_capacity=len(sids) // 2, max_batch=len(sids) + 3)
    gid = ctx.add_grammar(g)
    # rows: every state, plus DEAD, plus two ids that do not exist
    sid_rows = np.array(sids + [0, g.n_states, -5], np.int32)
    gid_rows = np.full(sid_rows.shape, gid, np.int32)
    B, W = sid_rows.size, dv.W
    for flags, stride in ((wg.WG_NO_CACHE, W), (wg.WG_USE_CACHE, W + 5), (wg.WG_USE_CACHE, W)):
        out = torch.full((B, stride), -1, dtype=torch.int32, device="cuda")
        wg.wg_build_masks(ctx, to_dev(torch, gid_rows), to_dev(torch, sid_rows), out[:, :W]
                          if stride == W else out, flags)
        got = out.cpu().numpy().view(np.uint32)
        assert (got[:len(sids), :W] == want).all(), (name, flags)
        assert (got[len(sids):, :W] == 0).all()
        if stride > W:
            assert (got[:, W:] == 0xFFFFFFFF).all(), "padding words were written"
    st = ctx.stats()
    assert st["bad_states"] >= 2 and st["rows_uncached"] > 0      # the pool held only half


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("V,pad", [(32000, 0), (32003, 0), (32003, 29), (40, 0), (1, 7), (70001, 15)])
def test_apply_and_argmax_match(wg, torch, dtype, V, pad):
    B = 7
    W = (V + 31) // 32
    rng = np.random.default_rng(V + pad)
    host = np.zeros((B, V + pad), np.float32 if dtype == "fp32" else np.uint16)
    host[:, :V] = make_logits(B, V, dtype, [5, V], 0)
    canary = 0x1234
    host[:, V:] = canary
    words = rng.integers(0, 1 << 32, size=(B, W), dtype=np.uint64).astype(np.uint32)
    words[0] = 0xFFFFFFFF
    words[1] = 0
    words[2] = 0
    words[2, W // 2] = 1 << 9 if V > (W // 2) * 32 + 9 else 1
    sparse = rng.random((W, 32)) < 0.01
    words[3] = np.packbits(sparse, axis=1, bitorder="little").view(np.uint32).ravel()
    dense = rng.random((W, 32)) < 0.97
    words[4] = np.packbits(dense, axis=1, bitorder="little").view(np.uint32).ravel()
    if V % 32:
        words[:, -1] &= (1 << (V % 32)) - 1
    want = host.copy()
    oracle.apply_mask(want, words, V)
    want_tok = oracle.argmax(host, words, V)
    raw_want = want.view(np.uint32) if dtype == "fp32" else want
    for with_argmax in (False, True):
        dl = dev_logits(torch, host, dtype)
        dm = to_dev(torch, words.view(np.int32))
        tok = torch.full((B,), -7, dtype=torch.int32, device="cuda") if with_argmax else None
        ws = torch.empty(wg.wg_apply_workspace_bytes(B), dtype=torch.uint8, device="cuda") \
            if with_argmax else None
        wg.wg_apply_mask(dl, dm, V, tok, ws)
        got = raw_bits(torch, dl)
        assert (got == raw_want).all(), (dtype, V, pad, with_argmax)
        if with_argmax:
            assert (tok.cpu().numpy() == want_tok).all()


def test_argmax_ties_and_signed_zero(wg, torch):
    V = 4096
    words = np.full((3, V // 32), 0xFFFFFFFF, np.uint32)
    words[:, 0] = 0xFFFFFFF0
    x = np.full((3, V), -1.0, np.float32)
    x[0, 2] = 9.0
    x[0, 1000] = -0.0
    x[0, 3000] = 0.0
    x[1, 777] = 0.5
    x[1, 4000] = 0.5
    x[2, :] = -np.inf
    want = oracle.argmax(x, words, V)
    assert want.tolist() == [1000, 777, 4]
    for dtype in ("fp32", "bf16"):
        host = x if dtype == "fp32" else (x.view(np.uint32) >> 16).astype(np.uint16)
        tok = torch.zeros(3, dtype=torch.int32, device="cuda")
        ws = torch.empty(wg.wg_apply_workspace_bytes(3), dtype=torch.uint8, device="cuda")
        wg.wg_apply_mask(dev_logits(torch, host, dtype), to_dev(torch, words.view(np.int32)), V, tok, ws)
        assert tok.cpu().tolist() == [1000, 777, 4]


class Sim:
    """One workload driven on both sides: same vocabulary, grammars, logits and tokens."""

    def __init__(self, wg, torch, vocab, ops, row_grammar, dtype, cache_capacity, use_cache=True,
                 seed=0, steer=6.0, delays=None, minimize=False, cache_mode=0, arena_bytes=0,
                 grams=None, starts=None, row_pad=0):
        self.wg, self.torch, self.vocab, self.dtype = wg, torch, vocab, dtype
        self.flats = [op if hasattr(op, "nodes") else flatten(op) for op in ops]
        self.trees = [oracle.Tree(f) for f in self.flats]
        # grams: library grammars made some other way than by lowering the trees (templates)
        self.grams = list(grams) if grams is not None else [wg.Grammar(f) for f in self.flats]
        if minimize:
            self.grams = [g.minimized() for g in self.grams]
        self.dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
        self.B = len(row_grammar)
        self.ctx = wg.Context(self.dv, cache_capacity, self.B, cache_mode, arena_bytes)
        self.gids = [self.ctx.add_grammar(g) for g in self.grams]
        self.row_grammar = list(row_grammar)
        self.flags = (wg.WG_USE_CACHE if use_cache else wg.WG_NO_CACHE) | wg.WG_RESTART_ON_DONE
        self.seed, self.steer = seed, steer
        self.row_pad = row_pad        # extra elements between logits rows (aligned rows, ragged V)
        self.bonus = has_structural_byte(vocab)
        self.delays = delays or [0] * self.B
        # a row that starts one step late sits in DONE first: it emits EOS and restarts
        late = [d > 0 for d in self.delays]
        # checker side
        self.cursors = [oracle.DONE if late[r] else self.trees[g].start()
                        for r, g in enumerate(self.row_grammar)]
        # library side
        self.d_gid = to_dev(torch, np.array([self.gids[g] for g in self.row_grammar], np.int32))
        self.d_sid = to_dev(torch, np.array(
            [self.grams[g].done_state if late[r] else self.grams[g].start_state
             for r, g in enumerate(self.row_grammar)], np.int32))
        if starts is not None:
            # rows that begin in the middle of a run: (library state, checker cursor) per row
            self.cursors = [c for _, c in starts]
            self.d_sid = to_dev(torch, np.array([s for s, _ in starts], np.int32))
        self.h_sid = self.d_sid.cpu().numpy().copy()
        self.W = self.dv.W
        self.d_mask = torch.zeros((self.B, self.W), dtype=torch.int32, device="cuda")
        self.d_tok = torch.zeros(self.B, dtype=torch.int32, device="cuda")
        self.d_status = torch.zeros(self.B, dtype=torch.int32, device="cuda")
        self.step_no = 0
        self.visited = set()

    def logits(self):
        x = make_logits(self.B, self.vocab.size, self.dtype, [self.seed, self.B], self.step_no,
                        self.bonus, self.steer)
        if any(self.delays) and self.step_no > 0:
            # a late row sees what the row before it saw one step earlier (kept on the device,
            # untouched by any kernel: a copy of the previous step's inputs)
            late = [r for r, d in enumerate(self.delays) if d > 0]
            idx = self.torch.tensor([r - 1 for r in late], device="cuda")
            bits = x.view(np.uint32) if self.dtype == "fp32" else x
            bits[late] = raw_bits(self.torch, self._prev_inputs[idx])
        return x

    def _remember_inputs(self, dl):
        if any(self.delays):
            self._prev_inputs = dl.clone()

    def step(self, check_rows=None, fused=True):
        wg, torch, vocab = self.wg, self.torch, self.vocab
        rows = range(self.B) if check_rows is None else check_rows
        host = self.logits()
        # ---- checker: mask -> apply -> argmax -> advance on the checked rows
        trees = [self.trees[self.row_grammar[r]] for r in rows]
        want_mask = oracle.masks(trees, vocab, [self.cursors[r] for r in rows],
                                 n_threads=oracle.max_threads())
        sub = np.ascontiguousarray(host[list(rows)])
        want_tok = oracle.argmax(sub, want_mask, vocab.size)
        want_logits = sub.copy()
        oracle.apply_mask(want_logits, want_mask, vocab.size)
        # ---- library
        dl = dev_logits(torch, host, self.dtype)
        if self.row_pad:
            wide = torch.zeros((self.B, vocab.size + self.row_pad), dtype=dl.dtype, device="cuda")
            wide[:, :vocab.size] = dl
            dl = wide[:, :vocab.size]
        self._remember_inputs(dl)
        if fused:
            wg.wg_decode_step(self.ctx, self.d_gid, self.d_sid, dl, self.d_mask, self.d_tok,
                              self.d_status, self.flags)
        else:
            ws = torch.empty(wg.wg_apply_workspace_bytes(self.B), dtype=torch.uint8, device="cuda")
            wg.wg_build_masks(self.ctx, self.d_gid, self.d_sid, self.d_mask, self.flags & 1)
            wg.wg_apply_mask(dl, self.d_mask, vocab.size, self.d_tok, ws)
            wg.wg_advance(self.ctx, self.d_gid, self.d_sid, self.d_tok, self.d_status,
                          self.flags & wg.WG_RESTART_ON_DONE)
        got_mask = self.d_mask.cpu().numpy().view(np.uint32)
        got_tok = self.d_tok.cpu().numpy()
        got_logits = raw_bits(torch, dl)
        got_sid = self.d_sid.cpu().numpy()
        status = self.d_status.cpu().numpy()
        raw_want = want_logits.view(np.uint32) if self.dtype == "fp32" else want_logits
        sel = list(rows)
        if not ((got_mask[sel] == want_mask).all() and (got_tok[sel] == want_tok).all()
                and (got_logits[sel] == raw_want).all() and (status[sel] == 0).all()):
            for i, r in enumerate(rows):          # name the first row that differs
                assert (got_mask[r] == want_mask[i]).all(), (self.step_no, r)
                assert got_tok[r] == want_tok[i], (self.step_no, r)
                assert (got_logits[r] == raw_want[i]).all(), (self.step_no, r)
                assert status[r] == 0
        # ---- advance the checker with the LIBRARY's tokens on every row (checked rows were
        # just shown to agree); unchecked rows are verified through the state mapping below
        for r in range(self.B):
            gi = self.row_grammar[r]
            t = int(got_tok[r])
            rc, cur = oracle.advance(self.trees[gi], vocab, self.cursors[r], t)
            assert rc == 0, (self.step_no, r, t)
            host_sid = self.grams[gi].step_token(int(self.h_sid[r]), t, token_symbols(vocab, t))
            if cur == oracle.DONE:
                cur = self.trees[gi].start()
                host_sid = self.grams[gi].start_state
            self.cursors[r] = cur
            assert got_sid[r] == host_sid, (self.step_no, r)
            self.visited.add((gi, host_sid))
        self.h_sid = got_sid.copy()
        self.step_no += 1

    def step_unchecked(self):
        """A step whose masks and logits are NOT compared: the logits are drawn on the device
        (seeded by the step number), so a long run between compared steps costs no host
        generation.  Every row is still checked through what is cheap: the library's token must
        be accepted by the checker in the row's cursor, and the device state must equal the host
        table walk of that token."""
        wg, torch, vocab = self.wg, self.torch, self.vocab
        if not hasattr(self, "_memo"):
            self._memo = {}
            self._bonus_dev = torch.from_numpy(self.bonus.astype(np.float32)).cuda() * self.steer
        gen = torch.Generator(device="cuda")
        gen.manual_seed(977 * self.seed + self.step_no)
        x = torch.randn((self.B, vocab.size), generator=gen, device="cuda") * 2.0
        if self.steer:
            x += self._bonus_dev
        dl = x.to(torch.bfloat16) if self.dtype == "bf16" else x
        if any(self.delays) and self.step_no > 0:
            late = [r for r, d in enumerate(self.delays) if d > 0]
            dl[late] = self._prev_inputs[torch.tensor([r - 1 for r in late], device="cuda")]
        self._remember_inputs(dl)
        wg.wg_decode_step(self.ctx, self.d_gid, self.d_sid, dl, self.d_mask, self.d_tok,
                          self.d_status, self.flags)
        got_tok = self.d_tok.cpu().numpy()
        got_sid = self.d_sid.cpu().numpy()
        assert (self.d_status == 0).all(), self.step_no
        for r in range(self.B):
            gi, t = self.row_grammar[r], int(got_tok[r])
            key = (gi, self.cursors[r], int(self.h_sid[r]), t)
            hit = self._memo.get(key)
            if hit is None:
                rc, cur = oracle.advance(self.trees[gi], vocab, self.cursors[r], t)
                assert rc == 0, (self.step_no, r, t)
                host_sid = self.grams[gi].step_token(int(self.h_sid[r]), t, token_symbols(vocab, t))
                if cur == oracle.DONE:
                    cur = self.trees[gi].start()
                    host_sid = self.grams[gi].start_state
                hit = self._memo[key] = (cur, host_sid)
            self.cursors[r] = hit[0]
            assert got_sid[r] == hit[1], (self.step_no, r)
            self.visited.add((gi, hit[1]))
        self.h_sid = got_sid.copy()
        self.step_no += 1


def test_trajectory_html_tiny(wg, torch):
    w = BY_NAME["html_tiny"]
    vocab = make_vocab(w.V, w.vocab_seed)
    sim = Sim(wg, torch, vocab, [w.grammar(0)], [0], w.dtype, cache_capacity=256, steer=8.0)
    for i in range(w.steps):                    # the workload's full 256 steps
        sim.step(fused=(i % 3 != 0))
    assert len(sim.visited) > 60
    st = sim.ctx.stats()
    assert st["cache_hits"] + st["cache_misses"] == w.steps and st["cache_hits"] > 0
    assert st["masks_built"] == st["cache_entries"] == st["cache_misses"]


def test_trajectory_json_lookup_batch32(wg, torch):
    w = BY_NAME["json_lookup"]
    vocab = make_vocab(w.V, w.vocab_seed)
    sim = Sim(wg, torch, vocab, [w.grammar(0)], [0] * 32, w.dtype, cache_capacity=2048, steer=6.0)
    for i in range(96):
        sim.step(check_rows=None if i < 4 else [0, 7, 31], fused=(i % 4 != 1))
    assert len(sim.visited) > 60


def test_cache_off_equals_cache_on_and_batch_order_does_not_matter(wg, torch):
    vocab = make_vocab(8192, seed=9)
    ops = [grammars.random_template(s) for s in range(3)]
    rows = [0, 1, 2, 0, 1, 2, 2, 2, 1, 0, 0]
    a = Sim(wg, torch, vocab, ops, rows, "bf16", cache_capacity=4096, use_cache=True, seed=3)
    b = Sim(wg, torch, vocab, ops, rows, "bf16", cache_capacity=0, use_cache=True, seed=3)
    c = Sim(wg, torch, vocab, ops, rows, "bf16", cache_capacity=4096, use_cache=False, seed=3)
    for _ in range(30):
        a.step()
        b.step()
        c.step()
        assert (a.d_mask == b.d_mask).all() and (a.d_mask == c.d_mask).all()
        assert (a.d_tok == c.d_tok).all()
    assert a.ctx.stats()["cache_hits"] > 0
    assert b.ctx.stats()["rows_uncached"] == 30 * len(rows)
    assert c.ctx.stats()["masks_built"] == 30 * len(rows)


def test_lookup_reports_slots_only_for_cached_states(wg, torch):
    vocab = make_vocab(4096, seed=4)
    g = wg.Grammar(flatten(grammars.html_template()))
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, cache_capacity=64, max_batch=16)
    gid = ctx.add_grammar(g)
    sid = to_dev(torch, np.array([1, 2, 3, 3, 2, 9, 1, 1], np.int32))
    gids = torch.full((8,), gid, dtype=torch.int32, device="cuda")
    slot = torch.zeros(8, dtype=torch.int32, device="cuda")
    wg.wg_mask_cache_lookup(ctx, gids, sid, slot)
    assert (slot.cpu().numpy() == -1).all()
    mask = torch.zeros((8, dv.W), dtype=torch.int32, device="cuda")
    wg.wg_build_masks(ctx, gids, sid, mask)
    wg.wg_mask_cache_lookup(ctx, gids, sid, slot)
    s = slot.cpu().numpy()
    assert (s >= 0).all() and len(set(s.tolist())) == 4
    assert s[0] == s[6] == s[7] and s[1] == s[4] and s[2] == s[3]
    st = ctx.stats()
    assert st["cache_entries"] == 4 and st["masks_built"] == 4
    assert st["cache_misses"] == 4 and st["cache_hits"] == 4
    ctx.cache_clear()
    wg.wg_mask_cache_lookup(ctx, gids, sid, slot)
    assert (slot.cpu().numpy() == -1).all()


def test_prewarm_caches_every_state_and_same_grammar_shares_an_id(wg, torch):
    vocab = make_vocab(6000, seed=6)
    flat = flatten(grammars.json_reference_lookup(doc_nodes=100))
    g1, g2 = wg.Grammar(flat), wg.Grammar(flat)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, cache_capacity=g1.n_states, max_batch=50)
    gid = ctx.add_grammar(g1)
    assert ctx.add_grammar(g2) == gid
    other = ctx.add_grammar(wg.Grammar(flatten(grammars.html_template())))
    assert other != gid
    ctx.cache_prewarm(gid)
    st = ctx.stats()
    assert st["cache_entries"] == g1.n_states - 1 == st["masks_built"]
    tree = oracle.Tree(flat)
    cursor_of = co_reachable(tree, g1, mentioned_symbols(flat))
    sids = sorted(cursor_of)[:50]
    mask = torch.zeros((len(sids), dv.W), dtype=torch.int32, device="cuda")
    wg.wg_build_masks(ctx, torch.full((len(sids),), gid, dtype=torch.int32, device="cuda"),
                      to_dev(torch, np.array(sids, np.int32)), mask)
    want = oracle.masks([tree] * len(sids), vocab, [cursor_of[s] for s in sids], n_threads=8)
    assert (mask.cpu().numpy().view(np.uint32) == want).all()
    assert ctx.stats()["masks_built"] == g1.n_states - 1       # nothing was rebuilt
    small = wg.Context(dv, cache_capacity=10, max_batch=50)
    sg = small.add_grammar(g1)
    with pytest.raises(wg.WgError) as e:
        small.cache_prewarm(sg)
    assert e.value.status == wg.binding.WG_ERR_CAPACITY


def test_advance_reports_rejected_tokens_and_keeps_the_state(wg, torch):
    vocab = make_vocab(4096, seed=4)
    flat = flatten(Sequence(Write(b"ab"), Wait(ALL_BYTES, SymSet(b";"))))
    g = wg.Grammar(flat)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, 0, 8)
    gid = ctx.add_grammar(g)
    tokens = np.array([ord("a"), ord("b"), vocab.size, -1, vocab.eos_id, ord("a"), ord("a")], np.int32)
    sids = np.array([1, 1, 1, 1, 1, 0, g.n_states + 4], np.int32)
    d_sid = to_dev(torch, sids)
    status = torch.zeros(7, dtype=torch.int32, device="cuda")
    wg.wg_advance(ctx, torch.full((7,), gid, dtype=torch.int32, device="cuda"), d_sid,
                  to_dev(torch, tokens), status)
    R, S = wg.binding.WG_ERR_TOKEN_REJECTED, wg.binding.WG_ERR_STATE
    assert status.cpu().tolist() == [0, R, R, R, R, R, S]
    assert d_sid.cpu().tolist() == [g.step(1, ord("a")), 1, 1, 1, 1, 0, g.n_states + 4]
    assert ctx.stats()["tokens_rejected"] == 5 and ctx.stats()["bad_states"] == 1


def test_empty_mask_gives_minus_one_and_an_error_status(wg, torch):
    # a vocabulary without the token the grammar needs next: nothing is allowed
    vocab = vocab_from_tokens([b"a", b"b", b"", b"c"] + [b"zz%d" % i for i in range(60)], eos_id=2)
    g = wg.Grammar(flatten(Write(b"Q")))
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, 4, 2)
    gid = ctx.add_grammar(g)
    d_sid = to_dev(torch, np.array([1, 1], np.int32))
    logits = torch.randn(2, vocab.size, device="cuda")
    mask = torch.zeros((2, dv.W), dtype=torch.int32, device="cuda")
    tok = torch.zeros(2, dtype=torch.int32, device="cuda")
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    wg.wg_decode_step(ctx, torch.full((2,), gid, dtype=torch.int32, device="cuda"), d_sid, logits,
                      mask, tok, status)
    assert tok.cpu().tolist() == [-1, -1]
    assert status.cpu().tolist() == [wg.binding.WG_ERR_EMPTY_MASK] * 2
    assert d_sid.cpu().tolist() == [1, 1]
    assert torch.isneginf(logits).all()


def test_host_argument_errors(wg, torch):
    vocab = make_vocab(1024, seed=4)
    with pytest.raises(wg.WgError):
        wg.Vocab(vocab.offsets, vocab.data, vocab.size)           # eos id out of range
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, 4, 4)
    five = torch.zeros(5, dtype=torch.int32, device="cuda")
    mask = torch.zeros((5, dv.W), dtype=torch.int32, device="cuda")
    with pytest.raises(wg.WgError) as e:                           # batch beyond max_batch
        wg.wg_build_masks(ctx, five, five, mask)
    assert e.value.status == wg.binding.WG_ERR_ARG
    narrow = torch.zeros((4, dv.W - 1), dtype=torch.int32, device="cuda")
    with pytest.raises(ValueError):                                # rows shorter than W words
        wg.wg_build_masks(ctx, five[:4], five[:4], narrow)
    with pytest.raises(wg.WgError):
        ctx.cache_prewarm(3)                                       # unknown grammar id


def test_trajectory_on_grammars_compiled_from_regular_expressions(wg, torch):
    from wg_workloads.optree import FlatTree
    patterns = [r"\[\d+(,\d+)*\]", r'\{"id": \d+, "tags": \[("[a-z]+"(, "[a-z]+")*)?\]\}',
                r"(yes|no|maybe)( \w+)*\."]
    flats = []
    for pat in patterns:
        t = wg.binding.RegexTree(pat)
        flats.append(FlatTree(t.nodes, t.children, t.sets, t.data, t.root))
    vocab = make_vocab(8192, seed=12)
    rows = [0, 1, 2, 0, 1, 2, 1, 1]
    sim = Sim(wg, torch, vocab, flats, rows, "fp32", cache_capacity=512, seed=8, steer=3.0)
    for _ in range(40):
        sim.step()
    assert len(sim.visited) > 25
    assert len({g for g, _ in sim.visited}) == 3


def test_host_buffer_step_and_step_plan_equal_the_plain_step(wg, torch):
    vocab = make_vocab(8192, seed=13)
    flat = flatten(grammars.json_reference_lookup(doc_nodes=60))
    g = wg.Grammar(flat)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    B, V = 6, vocab.size
    results = []
    for mode, cache_mode in (("plain", 0), ("plan", 0), ("host", 0), ("graph", 0), ("plain", 1),
                             ("graph", 1), ("host", 1)):
        ctx = wg.Context(dv, 256, B, cache_mode)
        gid = torch.full((B,), ctx.add_grammar(g), dtype=torch.int32, device="cuda")
        sid = torch.full((B,), g.start_state, dtype=torch.int32, device="cuda")
        mask = torch.zeros((B, dv.W), dtype=torch.int32, device="cuda")
        tok = torch.zeros(B, dtype=torch.int32, device="cuda")
        status = torch.zeros(B, dtype=torch.int32, device="cuda")
        plan = wg.StepPlan(ctx, gid, sid, mask, tok, status, wg.WG_RESTART_ON_DONE)
        tok_host = torch.zeros(B, dtype=torch.int32).pin_memory()
        fixed = torch.empty((B, V), dtype=torch.float32, device="cuda")
        graph = wg.StepGraph(ctx, gid, sid, fixed, mask, tok, status, wg.WG_RESTART_ON_DONE) \
            if mode == "graph" else None
        trace = []
        for step in range(25):
            host = torch.from_numpy(make_logits(B, V, "fp32", [3, 1], step))
            dl = host.cuda()
            if mode == "plain":
                wg.wg_decode_step(ctx, gid, sid, dl, mask, tok, status, wg.WG_RESTART_ON_DONE)
            elif mode == "plan":
                plan(dl)
            elif mode == "graph":
                fixed.copy_(dl)
                graph.launch()
                dl = fixed
            else:
                stage = torch.empty((B, V), dtype=torch.float32, device="cuda")
                wg.wg_decode_step_host(ctx, gid, sid, host.pin_memory(), stage, mask, tok, tok_host,
                                       status, wg.WG_RESTART_ON_DONE)
                assert (tok_host == tok.cpu()).all()
                dl = stage
            trace.append((tok.cpu().numpy().copy(), sid.cpu().numpy().copy(),
                          mask.cpu().numpy().copy(), dl.cpu().numpy().view(np.uint32).copy()))
            assert (status == 0).all()
        results.append(trace)
    for a, b in zip(results[0], results[1]):
        assert all((x == y).all() for x, y in zip(a, b))
    for other in results[2:]:
        for a, b in zip(results[0], other):
            assert all((x == y).all() for x, y in zip(a, b))


def test_degenerate_vocabularies_and_full_batches(wg, torch):
    # one-token vocabulary (the EOS token alone), very long tokens, a batch of exactly max_batch
    lone = vocab_from_tokens([b""], eos_id=0)
    g = wg.Grammar(flatten(Write(b"")))
    dv = wg.Vocab(lone.offsets, lone.data, 0)
    ctx = wg.Context(dv, 4, 3)
    gid = torch.full((3,), ctx.add_grammar(g), dtype=torch.int32, device="cuda")
    sid = torch.full((3,), g.start_state, dtype=torch.int32, device="cuda")
    mask = torch.zeros((3, 1), dtype=torch.int32, device="cuda")
    tok = torch.full((3,), 9, dtype=torch.int32, device="cuda")
    logits = torch.zeros((3, 8), device="cuda")[:, :1]          # V = 1, rows 32 bytes apart
    wg.wg_decode_step(ctx, gid, sid, logits, mask, tok)
    assert mask.cpu().tolist() == [[1]] * 3 and tok.cpu().tolist() == [0] * 3
    assert sid.cpu().tolist() == [g.done_state] * 3

    long_tokens = [b"ab" * 200, b"ab" * 127 + b"a", b"ab" * 200 + b"c", b"", b"a" * 255, b"a" * 256,
                   b"b" + b"a" * 300]
    vocab = vocab_from_tokens(long_tokens, eos_id=3)
    op = Sequence(Wait(SymSet(b"ab"), SymSet(b"c")), Write(b"!"))
    tree = oracle.Tree(flatten(op))
    g = wg.Grammar(flatten(op))
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, 0, 2)
    out = torch.zeros((2, 1), dtype=torch.int32, device="cuda")
    wg.wg_build_masks(ctx, torch.full((2,), ctx.add_grammar(g), dtype=torch.int32, device="cuda"),
                      torch.tensor([g.start_state, g.step(g.start_state, ord("c"))],
                                   dtype=torch.int32, device="cuda"), out, wg.WG_NO_CACHE)
    want = oracle.masks([tree, tree], vocab, [tree.start(), tree.step(tree.start(), ord("c"))])
    assert (out.cpu().numpy().view(np.uint32) == want).all()
    assert want[0, 0] == 0b1110111 and want[1, 0] == 0


def test_trajectory_with_token_level_writes(wg, torch):
    vocab = make_vocab(8192, seed=14)
    toks = vocab.tokens()
    forced = [toks.index(b"<"), 700, 701, vocab.eos_id, 5000]
    digits = SymSet(b"0123456789")
    loop = DoWhile(Sequence(WriteTokens([900, 901]), Wait(digits, digits)),
                   Cond(digits | b",;", SymSet(b","), SymSet(b";")))
    ops = [Sequence(Write(b"ab"), WriteTokens(forced), Write(b"cd"), loop),
           Sequence(WriteTokens([1, 3]), Wait(ALL_BYTES, SymSet(b"<")), WriteTokens([4000]))]
    sim = Sim(wg, torch, vocab, ops, [0, 1, 0, 0], "bf16", cache_capacity=256, seed=11, steer=4.0)
    for _ in range(60):
        sim.step(fused=(sim.step_no % 2 == 0))
    assert len(sim.visited) > 12
    # states of a token-level Write allow exactly their token
    g = sim.grams[0]
    forced_states = [s for s in range(1, g.n_states) if g.forced_token(s)]
    assert len(forced_states) == len(forced) + 2
    B = len(forced_states)
    out = torch.zeros((B, sim.dv.W), dtype=torch.int32, device="cuda")
    ctx = wg.Context(sim.dv, 0, B)
    wg.wg_build_masks(ctx, torch.full((B,), ctx.add_grammar(g), dtype=torch.int32, device="cuda"),
                      to_dev(torch, np.array(forced_states, np.int32)), out, wg.WG_NO_CACHE)
    bits = np.unpackbits(out.cpu().numpy().view(np.uint8), axis=1, bitorder="little")
    assert (bits.sum(axis=1) == 1).all()
    assert sorted(int(np.flatnonzero(b)[0]) for b in bits) == sorted(forced + [900, 901])


def test_forced_token_beyond_the_vocabulary_gives_an_empty_mask(wg, torch):
    vocab = make_vocab(1024, seed=14)
    g = wg.Grammar(flatten(WriteTokens([vocab.size + 7])))
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, 4, 1)
    gid = torch.full((1,), ctx.add_grammar(g), dtype=torch.int32, device="cuda")
    sid = torch.full((1,), g.start_state, dtype=torch.int32, device="cuda")
    mask = torch.ones((1, dv.W), dtype=torch.int32, device="cuda")
    tok = torch.zeros(1, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    wg.wg_decode_step(ctx, gid, sid, torch.zeros((1, vocab.size), device="cuda"), mask, tok, status)
    assert (mask == 0).all() and tok.item() == -1
    assert status.item() == wg.binding.WG_ERR_EMPTY_MASK and sid.item() == g.start_state


@pytest.mark.parametrize("B", [3000, 20000])      # several passes of the one-block lookup kernel
def test_large_batch_stats_reset_and_kernel_timing(wg, torch, B):
    vocab = make_vocab(2048, seed=15)
    flat = flatten(grammars.json_reference_lookup(doc_nodes=40))
    tree, g = oracle.Tree(flat), wg.Grammar(flat)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, 512, B)
    gid = torch.full((B,), ctx.add_grammar(g), dtype=torch.int32, device="cuda")
    cursor_of = co_reachable(tree, g, mentioned_symbols(flat))
    sids = sorted(cursor_of)
    rows = np.array([sids[(7 * r) % len(sids)] for r in range(B)], np.int32)
    sid = to_dev(torch, rows)
    mask = torch.zeros((B, dv.W), dtype=torch.int32, device="cuda")
    tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(B, dtype=torch.int32, device="cuda")
    host = make_logits(B, vocab.size, "bf16", [15, 0], 0)
    want_masks = {s: oracle.mask(tree, vocab, cursor_of[s]) for s in set(rows.tolist())}
    ctx.set_timing(True)
    wg.wg_decode_step(ctx, gid, sid, dev_logits(torch, host, "bf16"), mask, tok, status)
    t = ctx.get_timing()
    assert t["steps"] == 1 and t["apply_ms"] > 0 and t["build_ms"] > 0
    assert ctx.get_timing()["steps"] == 0             # reading forgets the recorded steps
    ctx.set_timing(False)
    got = mask.cpu().numpy().view(np.uint32)
    want = np.stack([want_masks[s] for s in rows.tolist()])
    assert (got == want).all()
    assert (tok.cpu().numpy() == oracle.argmax(host, want, vocab.size)).all()
    st = ctx.stats()
    assert st["cache_misses"] == len(set(rows.tolist())) == st["masks_built"]
    assert st["cache_hits"] == B - st["cache_misses"]
    ctx.reset_stats()
    assert all(v == 0 for k, v in ctx.stats().items() if k not in ("cache_entries", "cache_bytes"))


def test_trajectory_on_minimized_grammars(wg, torch):
    vocab = make_vocab(8192, seed=16)
    ops = [grammars.json_reference_lookup(doc_nodes=200), grammars.dynamic_snippet_template(1, n_args=3, enum_size=12)]
    sim = Sim(wg, torch, vocab, ops, [0, 1, 0, 1, 0], "bf16", cache_capacity=1024, seed=9, steer=5.0,
              minimize=True)
    assert sim.grams[0].n_states < wg.Grammar(sim.flats[0]).n_states
    for _ in range(50):
        sim.step()
    assert len(sim.visited) > 30


def test_masks_of_random_trees_on_a_dense_small_alphabet_vocabulary(wg, torch):
    import itertools
    from test_oracle_pins import _random_tree
    rng = np.random.default_rng(31)
    alphabet = b"abcd,;"
    tokens = [b""]                                                   # id 0 = EOS
    for n in (1, 2, 3):
        tokens += [bytes(t) for t in itertools.product(alphabet, repeat=n)]
    tokens += [bytes(rng.choice(list(alphabet), size=int(rng.integers(4, 24))).tolist())
               for _ in range(900)]
    tokens += [b"x", b"ax", b""]
    vocab = vocab_from_tokens(tokens, eos_id=0)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    symbols = list(alphabet) + [ord("x"), EOS]
    ctx = wg.Context(dv, 4096, 512)
    n_states = 0
    for _ in range(25):
        flat = flatten(_random_tree(rng, 3))
        tree, g = oracle.Tree(flat), wg.Grammar(flat)
        cursor_of = co_reachable(tree, g, symbols)
        sids = sorted(cursor_of)[:512]
        gid = ctx.add_grammar(g)
        want = oracle.masks([tree] * len(sids), vocab, [cursor_of[s] for s in sids], n_threads=8)
        for flags in (wg.WG_NO_CACHE, wg.WG_USE_CACHE):
            out = torch.zeros((len(sids), dv.W), dtype=torch.int32, device="cuda")
            wg.wg_build_masks(ctx, torch.full((len(sids),), gid, dtype=torch.int32, device="cuda"),
                              to_dev(torch, np.array(sids, np.int32)), out, flags)
            assert (out.cpu().numpy().view(np.uint32) == want).all()
        n_states += len(sids)
    assert n_states > 150


def test_bad_state_ids_take_no_cache_entry_and_are_counted_every_step(wg, torch):
    vocab = make_vocab(4096, seed=4)
    g = wg.Grammar(flatten(grammars.html_template()))
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, cache_capacity=64, max_batch=4)
    gid = torch.full((3,), ctx.add_grammar(g), dtype=torch.int32, device="cuda")
    sid = to_dev(torch, np.array([g.start_state, g.n_states + 3, -9], np.int32))
    mask = torch.ones((3, dv.W), dtype=torch.int32, device="cuda")
    tok = torch.zeros(3, dtype=torch.int32, device="cuda")
    status = torch.zeros(3, dtype=torch.int32, device="cuda")
    for step in range(2):
        logits = torch.randn(3, vocab.size, device="cuda")
        wg.wg_decode_step(ctx, gid, sid.clone(), logits, mask, tok, status)
        assert (mask[1:] == 0).all() and tok.cpu().tolist()[1:] == [-1, -1]
        assert status.cpu().tolist()[1:] == [wg.binding.WG_ERR_STATE] * 2
    st = ctx.stats()
    # two bad rows a step: counted when their zero masks are built and again by the advance
    assert st["bad_states"] == 2 * 2 * 2 and st["cache_entries"] == 1
    assert st["rows_uncached"] == 4 and st["cache_hits"] == 1


def test_equal_tables_over_different_class_maps_are_different_grammars(wg, torch):
    vocab = make_vocab(1024, seed=4)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    ctx = wg.Context(dv, 16, 2)
    ga, gb = wg.Grammar(flatten(Write(b"a"))), wg.Grammar(flatten(Write(b"b")))
    ida, idb = ctx.add_grammar(ga), ctx.add_grammar(gb)
    assert ida != idb and ctx.add_grammar(wg.Grammar(flatten(Write(b"a")))) == ida
    out = torch.zeros((2, dv.W), dtype=torch.int32, device="cuda")
    wg.wg_build_masks(ctx, to_dev(torch, np.array([ida, idb], np.int32)),
                      to_dev(torch, np.array([ga.start_state, gb.start_state], np.int32)), out)
    bits = np.unpackbits(out.cpu().numpy().view(np.uint8), axis=1, bitorder="little")
    assert np.flatnonzero(bits[0]).tolist() == [ord("a")]
    assert np.flatnonzero(bits[1]).tolist() == [ord("b")]


@pytest.mark.parametrize("cache_mode,capacity,arena", [(0, 3, 0), (0, 40, 0), (1, 40, 4096), (1, 6, 0)])
def test_one_launch_step_with_a_cache_that_fills_up(wg, torch, cache_mode, capacity, arena):
    """Small batches take the one-launch step, which files new masks itself.  A pool (or a compact
    arena) that is too small must leave the later states uncached -- built on every visit, with
    the same masks, tokens and states as ever."""
    vocab = make_vocab(8192, seed=17)
    ops = [grammars.html_template(), grammars.json_reference_lookup(doc_nodes=60)]
    rows = [0, 1, 1, 0, 1, 0, 1]
    sim = Sim(wg, torch, vocab, ops, rows, "bf16", cache_capacity=capacity, seed=12, steer=6.0,
              cache_mode=cache_mode, arena_bytes=arena)
    for _ in range(60):
        sim.step()
    st = sim.ctx.stats()
    assert len(sim.visited) > capacity, "the run must meet more states than the cache holds"
    assert st["rows_uncached"] > 0 and st["cache_entries"] <= capacity
    assert st["cache_hits"] + st["cache_misses"] == 60 * len(rows)
    assert st["masks_built"] >= st["cache_misses"] - 0 and st["cache_hits"] > 0


def test_one_launch_step_at_its_largest_batch_and_the_first_batch_beyond(wg, torch):
    vocab = make_vocab(8192, seed=18)
    ops = [grammars.json_reference_lookup(doc_nodes=80), grammars.random_template(5)]
    for B in (64, 65):
        rows = [r % 2 for r in range(B)]
        sim = Sim(wg, torch, vocab, ops, rows, "fp32", cache_capacity=1024, seed=B, steer=5.0)
        launches = wg.kernel_launch_count()
        for _ in range(12):
            sim.step()
        per_step = (wg.kernel_launch_count() - launches) / 12
        assert per_step == (1 if B == 64 else 4)
        assert sim.ctx.stats()["rows_uncached"] == 0 and len(sim.visited) > 10


def test_batches_beyond_the_row_limit_are_refused(wg, torch):
    vocab = make_vocab(1024, seed=4)
    dv = wg.Vocab(vocab.offsets, vocab.data, vocab.eos_id)
    with pytest.raises(wg.WgError) as e:
        wg.Context(dv, 4, 65536)                   # WG_MAX_ROWS is 65535
    assert e.value.status == wg.binding.WG_ERR_ARG
    wg.Context(dv, 4, 65535).close()


def test_one_launch_step_on_random_trees_with_a_dense_small_alphabet_vocabulary(wg, torch):
    """The in-kernel mask build of the one-launch step on grammars nobody designed: random operator
    trees over a six-letter alphabet and a vocabulary that holds every string of up to three
    letters, so that most tokens are decided by the walk and many survive it."""
    import itertools
    from test_oracle_pins import _random_tree
    rng = np.random.default_rng(41)
    alphabet = b"abcd,;"
    tokens = [b""]                                                   # id 0 = EOS
    for n in (1, 2, 3):
        tokens += [bytes(t) for t in itertools.product(alphabet, repeat=n)]
    tokens += [bytes(rng.choice(list(alphabet), size=int(rng.integers(4, 24))).tolist())
               for _ in range(1500)]
    vocab = vocab_from_tokens(tokens, eos_id=0)
    n_visited = 0
    for _ in range(12):
        ops = [_random_tree(rng, 3) for _ in range(3)]
        rows = [0, 1, 2, 0, 1, 2, 2, 1, 0]
        for cache_mode in (0, 1):
            sim = Sim(wg, torch, vocab, ops, rows, "fp32", cache_capacity=256, seed=int(rng.integers(1 << 20)),
                      steer=0.0, cache_mode=cache_mode)
            for _ in range(10):
                sim.step()
            n_visited += len(sim.visited)
    assert n_visited > 150


def test_one_launch_step_when_a_warp_queues_more_tokens_than_its_queue_holds(wg, torch):
    """At 64 rows and more than about 600 000 tokens a warp of the one-launch step takes two spans
    at a time.  In a state that leaves on any of forty bytes every token is walked, 2 048 per warp
    and pass, more than the warp's queue of 1 024 holds: the spans are then walked one by one."""
    vocab = make_vocab(620000, seed=19)
    leaving = SymSet(b"0123456789abcdefghijklmnopqrstuvwxyzABCD")
    op = Sequence(Wait(allow=ALL_BYTES, wait=leaving), Write(b"!"), Wait(allow=ALL_BYTES, wait=SymSet(b"<")))
    B = 64
    sim = Sim(wg, torch, vocab, [op], [0] * B, "fp32", cache_capacity=0, use_cache=False, seed=23, steer=0.0)
    launches = wg.kernel_launch_count()
    for _ in range(2):
        sim.step()
    assert wg.kernel_launch_count() - launches == 2          # the one-launch step
    assert sim.ctx.stats()["masks_built"] == 2 * B


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_one_launch_step_on_a_vocabulary_whose_size_is_no_multiple_of_anything(wg, torch, dtype):
    vocab = odd_vocab()                      # V % 32 != 0, V % 8 != 0: ragged last word and chunk
    assert vocab.size % 8 != 0
    ops = [grammars.html_template(), grammars.json_reference_lookup(doc_nodes=60)]
    pad = 16 - vocab.size % 16               # rows 32 or 64 bytes apart modulo 16: aligned rows
    sim = Sim(wg, torch, vocab, ops, [0, 1, 0, 1, 1], dtype, cache_capacity=512, seed=31, steer=6.0,
              row_pad=pad)
    launches = wg.kernel_launch_count()
    for _ in range(40):
        sim.step()
    assert wg.kernel_launch_count() - launches == 40          # aligned rows: the one-launch step
    assert len(sim.visited) > 30 and sim.ctx.stats()["cache_hits"] > 0


@pytest.mark.parametrize("B,dtype,cache_mode,use_cache", [(5, "fp32", 0, True), (96, "bf16", 0, True),
                                                          (96, "bf16", 1, True), (70, "fp32", 0, False)])
def test_mask_only_step_for_an_engine_that_samples_itself(wg, torch, B, dtype, cache_mode, use_cache):
    """wg_decode_step without token_out: masks and masked logits as the checker's, states left
    alone; the test then "samples" a random allowed token per row and hands it to wg_advance."""
    vocab = make_vocab(12000 + 7, seed=41)
    ops = [grammars.html_template(), grammars.json_reference_lookup(doc_nodes=60)]
    rows = [r % 2 for r in range(B)]
    sim = Sim(wg, torch, vocab, ops, rows, dtype, cache_capacity=2048, seed=B, steer=4.0,
              cache_mode=cache_mode, use_cache=use_cache)
    rng = np.random.default_rng(B)
    flags = wg.WG_USE_CACHE if use_cache else wg.WG_NO_CACHE
    V = vocab.size
    for step in range(40):
        host = sim.logits()
        trees = [sim.trees[g] for g in rows]
        want_mask = oracle.masks(trees, vocab, sim.cursors, n_threads=oracle.max_threads())
        want_logits = host.copy()
        oracle.apply_mask(want_logits, want_mask, V)
        dl = dev_logits(torch, host, dtype)
        before = sim.d_sid.clone()
        wg.wg_decode_step(sim.ctx, sim.d_gid, sim.d_sid, dl, sim.d_mask, None, None, flags)
        assert (sim.d_sid == before).all(), "a step that chooses no token advances nothing"
        got_mask = sim.d_mask.cpu().numpy().view(np.uint32)
        assert (got_mask == want_mask).all(), step
        raw_want = want_logits.view(np.uint32) if dtype == "fp32" else want_logits
        assert (raw_bits(torch, dl) == raw_want).all(), step
        # the engine's sampler: any allowed token
        bits = np.unpackbits(want_mask.view(np.uint8), axis=1, bitorder="little")[:, :V]
        toks = np.array([rng.choice(np.flatnonzero(bits[r])) for r in range(B)], np.int32)
        d_tok = to_dev(torch, toks)
        wg.wg_advance(sim.ctx, sim.d_gid, sim.d_sid, d_tok, sim.d_status, wg.WG_RESTART_ON_DONE)
        assert (sim.d_status.cpu().numpy() == 0).all()
        got_sid = sim.d_sid.cpu().numpy()
        for r in range(B):
            gi, t = rows[r], int(toks[r])
            rc, cur = oracle.advance(sim.trees[gi], vocab, sim.cursors[r], t)
            assert rc == 0
            host_sid = sim.grams[gi].step_token(int(sim.h_sid[r]), t, token_symbols(vocab, t))
            if cur == oracle.DONE:
                cur, host_sid = sim.trees[gi].start(), sim.grams[gi].start_state
            sim.cursors[r] = cur
            assert got_sid[r] == host_sid, (step, r)
            sim.visited.add((gi, host_sid))
        sim.h_sid = got_sid.copy()
        sim.step_no += 1
    assert len(sim.visited) > 40
    with pytest.raises(ValueError):                 # nothing advances: a status array has no meaning
        wg.wg_decode_step(sim.ctx, sim.d_gid, sim.d_sid, dl, sim.d_mask, None, sim.d_status, flags)
    with pytest.raises(ValueError):
        wg.wg_decode_step(sim.ctx, sim.d_gid, sim.d_sid, dl, sim.d_mask, None, None,
                          flags | wg.WG_RESTART_ON_DONE)
