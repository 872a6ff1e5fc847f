"""The allocation-free mask + argmax entry point against the ordinary one.

Some users of the library cannot allocate device memory at the point where they mask logits
(a server whose memory pool owns the whole GPU, code running inside another framework's step
where an allocation would stall the device).  ``wg_apply_mask_noalloc`` serves them with a
fixed scratch array inside the library.  This file checks, through the C ABI, that it gives
bit-identical logits and tokens to ``wg_apply_mask`` on two calls in a row (the second call
sees the first call's leftovers in the shared scratch and must not be disturbed by them) and
that it refuses batches beyond its fixed size.  It is collected last on purpose.
"""
import numpy as np
import pytest

from wg_workloads import make_logits

pytestmark = pytest.mark.gpu


def _case(rng, B, V, dtype, seed):
    W = (V + 31) // 32
    host = make_logits(B, V, dtype, [seed, V], 0)
    words = rng.integers(0, 1 << 32, size=(B, W), dtype=np.uint64).astype(np.uint32)
    words[0] = 0
    words[0, W // 3] = 1 << 5
    sparse = rng.random((B // 2, W, 32)) < 0.02
    words[1:1 + B // 2] = np.packbits(sparse, axis=2, bitorder="little").view(np.uint32).reshape(B // 2, W)
    if V % 32:
        words[:, -1] &= (1 << (V % 32)) - 1
    return host, words


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_noalloc_matches_apply_mask_on_two_calls_in_a_row(dtype):
    import torch

    import paper_2507_16768_b200 as wg

    torch.cuda.set_device(0)
    rng = np.random.default_rng(123)
    # the second call is smaller and has different winners: stale maxima of the first call
    # sit in the rows it reuses and in the rows it does not touch
    for B, V, seed in ((96, 128256, 1), (17, 40000, 2)):
        host, words = _case(rng, B, V, dtype, seed)

        def upload():
            if dtype == "bf16":
                return torch.from_numpy(host.view(np.int16)).cuda().view(torch.bfloat16)
            return torch.from_numpy(host).cuda()

        mask = torch.from_numpy(words.view(np.int32)).cuda()
        ref_logits, ref_tok = upload(), torch.full((B,), -9, dtype=torch.int32, device="cuda")
        ws = torch.empty(wg.wg_apply_workspace_bytes(B), dtype=torch.uint8, device="cuda")
        wg.wg_apply_mask(ref_logits, mask, V, ref_tok, ws)
        got_logits, got_tok = upload(), torch.full((B,), -9, dtype=torch.int32, device="cuda")
        wg.wg_apply_mask_noalloc(got_logits, mask, V, got_tok)
        torch.cuda.synchronize()
        assert torch.equal(got_tok, ref_tok)
        as_int = torch.int16 if dtype == "bf16" else torch.int32
        assert torch.equal(got_logits.view(as_int), ref_logits.view(as_int))
        assert (ref_tok >= 0).all()


def test_noalloc_rejects_batches_beyond_its_fixed_scratch():
    import torch

    import paper_2507_16768_b200 as wg

    torch.cuda.set_device(0)
    B, V = wg.binding.WG_NOALLOC_MAX_ROWS + 1, 64
    logits = torch.zeros((B, V), device="cuda")
    mask = torch.full((B, 2), -1, dtype=torch.int32, device="cuda")
    tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    with pytest.raises(wg.WgError) as e:
        wg.wg_apply_mask_noalloc(logits, mask, V, tok)
    assert e.value.status == wg.binding.WG_ERR_CAPACITY
    assert (logits == 0).all()                      # nothing ran
    wg.wg_apply_mask_noalloc(logits[:-1], mask[:-1], V, tok[:-1])   # exactly the maximum is fine
    torch.cuda.synchronize()
    assert (tok[:-1] == 0).all()
