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
