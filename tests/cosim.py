"""Drives the CPU checker and the library side by side over the same symbols / tokens."""
from __future__ import annotations

from collections import deque
from typing import Dict, Iterable, List, Tuple

import numpy as np

import oracle
from wg_workloads import EOS, flatten


def mentioned_symbols(flat) -> List[int]:
    """Symbols that occur in any set or literal of the tree, plus a few that do not."""
    syms = set(int(b) for b in flat.data)
    bits = np.bitwise_or.reduce(flat.sets, axis=0) if flat.sets.shape[0] else np.zeros(9, np.uint32)
    all_and = np.bitwise_and.reduce(flat.sets, axis=0) if flat.sets.shape[0] else bits
    for s in range(257):
        in_some = (int(bits[s >> 5]) >> (s & 31)) & 1
        in_all = (int(all_and[s >> 5]) >> (s & 31)) & 1
        if in_some and not in_all:
            syms.add(s)
    # symbols the sets treat alike still need a few representatives
    for extra in (0, ord(" "), ord("a"), ord("Z"), ord("5"), ord("<"), ord('"'), 0x7F, 0xC3, 0xFF, EOS):
        syms.add(extra)
    return sorted(syms)


def symbol_representatives(flat) -> List[int]:
    """One symbol of every group of symbols that the tree cannot tell apart.

    Two symbols are told apart when some set of the tree holds one and not the other, or when
    one of them is a byte of a literal.  This is a property of the input arrays alone."""
    member = np.zeros((flat.sets.shape[0] + 1, 257), np.uint8)
    for s in range(257):
        member[:-1, s] = (flat.sets[:, s >> 5] >> np.uint32(s & 31)) & 1
    member[-1, :] = 0
    literal = np.unique(np.asarray(flat.data, np.uint8))
    seen, reps = set(), []
    sig = np.packbits(member, axis=0)
    in_literal = np.zeros(257, bool)
    in_literal[literal] = True
    for s in range(257):
        key = (bytes(sig[:, s]), s if (in_literal[s] or s == EOS) else -1)   # end-of-sequence stands alone
        if key not in seen:
            seen.add(key)
            reps.append(s)
    return reps


def co_reachable(tree: oracle.Tree, grammar, symbols: Iterable[int], max_states: int = 10 ** 9
                 ) -> Dict[int, Tuple[int, int]]:
    """Breadth-first walk of both automata with the same symbols.

    Checks that every transition agrees on DEAD / not DEAD and that a checker cursor always
    lands on the same library state.  Returns {library state: one checker cursor}.
    """
    symbols = list(symbols)
    start = tree.start()
    sid_of = {start: grammar.start_state}
    cursor_of = {grammar.start_state: start}
    queue = deque([start])
    while queue and len(cursor_of) < max_states:
        cur = queue.popleft()
        sid = sid_of[cur]
        for s in symbols:
            nxt = tree.step(cur, s)
            nsid = grammar.step(sid, s)
            assert oracle.is_dead(nxt) == (nsid == 0), (cur, sid, s)
            if nsid == 0:
                continue
            if nxt in sid_of:
                assert sid_of[nxt] == nsid, (cur, s, nxt)
                continue
            sid_of[nxt] = nsid
            if nsid not in cursor_of:
                cursor_of[nsid] = nxt
            queue.append(nxt)
    return cursor_of


def token_symbols(vocab, t: int) -> List[int]:
    return [EOS] if t == vocab.eos_id else list(vocab.token(t))


def random_walk_states(tree: oracle.Tree, grammar, symbols: Iterable[int], rng, n_walks: int,
                       max_steps: int) -> Dict[int, Tuple[int, int]]:
    """States met on random walks of both automata from the start (for grammars too large to
    enumerate).  At each step one of the symbols that keeps both sides alive is taken, so a walk
    runs deep into the grammar; a finished walk starts again.  Returns {library state: cursor}."""
    symbols = list(symbols)
    cursor_of = {grammar.start_state: tree.start()}
    for _ in range(n_walks):
        cur, sid = tree.start(), grammar.start_state
        for _ in range(max_steps):
            live = []
            for s in symbols:
                nsid = grammar.step(sid, s)
                if nsid != 0:
                    live.append((s, nsid))
            if not live:
                break
            s, nsid = live[int(rng.integers(0, len(live)))]
            cur = tree.step(cur, s)
            assert not oracle.is_dead(cur), (sid, s)
            if cur == oracle.DONE:
                break
            sid = nsid
            cursor_of.setdefault(sid, cur)
    return cursor_of
