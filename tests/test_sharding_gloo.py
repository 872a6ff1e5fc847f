"""World-size-2 check of the multi-GPU host logic on CPU (gloo): rows split across ranks give
the same masks and tokens as one rank doing the whole batch, and the job time is the slowest
rank's.  The per-row work here is done by the CPU checker; on GPUs each rank would call the
library on its slice in exactly the same way."""
import os
import socket

import numpy as np
import pytest


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str) -> None:
    import torch
    import torch.distributed as dist

    import oracle
    from paper_2507_16768_b200.sharding import (gather_tokens, max_over_ranks, reduce_best_keys,
                                                shard_rows, vocab_slices)
    from wg_workloads import flatten, grammars, make_logits, make_vocab

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n_rows = 7
        vocab = make_vocab(3000, seed=8)
        tree = oracle.Tree(flatten(grammars.json_reference_lookup(doc_nodes=0)))
        prefixes = [b"[", b'[{"topic": ', b'[{"topic": 4', b'[{"topic": 41, "paths": ["',
                    b'[{"topic": 7, "paths": ["12', b'[{"topic": 7, "paths": ["12/3"',
                    b'[{"topic": 7, "paths": ["1"]}']
        cursors = [tree.walk(tree.start(), list(p)) for p in prefixes]
        logits = make_logits(n_rows, vocab.size, "fp32", 5)
        b, e = shard_rows(n_rows, world, rank)
        masks = oracle.masks([tree] * (e - b), vocab, cursors[b:e])
        tok = oracle.argmax(np.ascontiguousarray(logits[b:e]), masks, vocab.size)
        everyone = gather_tokens(torch.from_numpy(tok), n_rows)
        slowest = max_over_ranks(10.0 + rank)
        # the vocabulary split: every rank takes all rows but only its token slice; the per-row
        # (value, token) pairs travel as one int64 each and the MAX all-reduce picks the winner
        vb, ve = vocab_slices(vocab.size, world, align=1024)[rank]
        all_masks = oracle.masks([tree] * n_rows, vocab, cursors)
        sliced = np.zeros_like(all_masks)
        for t in range(vb, ve):
            sliced[:, t >> 5] |= all_masks[:, t >> 5] & np.uint32(1 << (t & 31))
        local = oracle.argmax(logits, sliced, vocab.size)          # best token inside the slice
        keys = torch.full((n_rows,), -(1 << 63), dtype=torch.int64)
        for r in range(n_rows):
            if local[r] >= 0:
                bits = int(np.float32(logits[r, local[r]]).view(np.uint32))
                if bits == 0x80000000:
                    bits = 0
                ordered = (~bits & 0xFFFFFFFF) if bits & 0x80000000 else (bits | 0x80000000)
                packed = (ordered << 32) | (0xFFFFFFFF - int(local[r]))
                keys[r] = (packed ^ (1 << 63)) - (1 << 64) if (packed ^ (1 << 63)) >= (1 << 63) \
                    else (packed ^ (1 << 63))
        reduce_best_keys(keys)
        winners = [0xFFFFFFFF - ((int(k) + (1 << 64)) & 0xFFFFFFFF) for k in keys.tolist()]
        if rank == 0:
            full_masks = oracle.masks([tree] * n_rows, vocab, cursors)
            assert winners == oracle.argmax(logits, full_masks, vocab.size).tolist()
            full_tok = oracle.argmax(logits, full_masks, vocab.size)
            assert everyone == full_tok.tolist()
            assert slowest == 10.0 + world - 1
            open(os.path.join(out_dir, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_shard_rows_tiles_the_batch():
    from paper_2507_16768_b200.sharding import shard_rows
    for n in (0, 1, 7, 1024, 1025):
        for world in (1, 2, 3, 8):
            spans = [shard_rows(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_rows(4, 2, 2)


def test_two_ranks_equal_one_rank(tmp_path):
    import torch.multiprocessing as mp
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").read_text() == "ok"


def test_vocab_slices_tile_the_vocabulary_on_aligned_boundaries():
    from paper_2507_16768_b200.sharding import vocab_slices
    for V in (1, 8192, 8193, 128256, 151936, 256000):
        for world in (1, 2, 3, 8):
            sl = vocab_slices(V, world)
            assert sl[0][0] == 0 and sl[-1][1] == V
            assert all(a[1] == b[0] for a, b in zip(sl, sl[1:]))
            assert all(b % 8192 == 0 and (e % 8192 == 0 or e == V) for b, e in sl if e > b)
            pieces = [(e - b + 8191) // 8192 for b, e in sl]
            assert max(pieces) - min(pieces) <= 1
