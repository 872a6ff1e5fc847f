"""The Python binding refuses arrays that the kernels would index out of bounds.

The kernels take raw pointers and index them by row number, so a short, strided or misplaced
array must be caught by the binding, before the library is called.  These tests run without a
GPU: the arrays are stand-ins with the attributes of CUDA tensors, and the library handle is
replaced by one that fails the test when any entry point is reached.
"""
import pytest
import torch

import paper_2507_16768_b200 as wg
from paper_2507_16768_b200 import binding


class FakeDevice:
    def __init__(self, index):
        self.index = index


class FakeTensor:
    """What the binding reads of a tensor: shape, strides, dtype, device."""

    def __init__(self, shape, dtype=torch.int32, device=0, strides=None, cuda=True):
        self.shape = tuple(shape)
        self.dtype = dtype
        self.is_cuda = cuda
        self.device = FakeDevice(device)
        if strides is None:
            strides, n = [], 1
            for d in reversed(self.shape):
                strides.insert(0, n)
                n *= d
        self._strides = tuple(strides)

    def dim(self):
        return len(self.shape)

    def stride(self, i):
        return self._strides[i]

    def numel(self):
        n = 1
        for d in self.shape:
            n *= d
        return n

    def element_size(self):
        return {torch.int32: 4, torch.int64: 8, torch.float32: 4, torch.bfloat16: 2,
                torch.uint8: 1}[self.dtype]

    def is_contiguous(self):
        n = 1
        for d, s in zip(reversed(self.shape), reversed(self._strides)):
            if s != n:
                return False
            n *= d
        return True

    def data_ptr(self):
        return 0x1000


class FakeVocab:
    V, W, device = 1000, 32, 0


class FakeContext:
    handle, vocab, device, max_batch = None, FakeVocab(), 0, 64


class Unreachable:
    def __getattr__(self, name):
        if name == "wg_apply_workspace_bytes":      # a size formula on the host, no device work
            return lambda rows: 8 * rows

        def entry(*args):
            raise AssertionError(f"{name} was called with arguments that must be refused")
        return entry


@pytest.fixture
def no_library(monkeypatch):
    monkeypatch.setattr(binding, "_lib", Unreachable())
    monkeypatch.setattr(binding, "_stream_ptr", lambda stream: None)


B, V, W = 8, FakeVocab.V, FakeVocab.W


def good():
    return dict(gid=FakeTensor([B]), sid=FakeTensor([B]), logits=FakeTensor([B, V], torch.float32),
                bitmask=FakeTensor([B, W]), token_out=FakeTensor([B]), status=FakeTensor([B]))


BAD = {
    "short gid": dict(gid=FakeTensor([B - 1])),
    "strided sid": dict(sid=FakeTensor([B], strides=[2])),
    "short token_out": dict(token_out=FakeTensor([B - 3])),
    "short status": dict(status=FakeTensor([1])),
    "bitmask with fewer rows": dict(bitmask=FakeTensor([B - 1, W])),
    "bitmask with fewer words": dict(bitmask=FakeTensor([B, W - 1])),
    "bitmask with a strided inner dimension": dict(bitmask=FakeTensor([B, W], strides=[2 * W, 2])),
    "logits with fewer columns than the vocabulary": dict(logits=FakeTensor([B, V - 1], torch.float32)),
    "gid on another device": dict(gid=FakeTensor([B], device=1)),
    "logits on another device": dict(logits=FakeTensor([B, V], torch.float32, device=1)),
    "2-D sid": dict(sid=FakeTensor([B, 1])),
}


@pytest.mark.parametrize("case", sorted(BAD))
def test_decode_step_refuses(no_library, case):
    a = {**good(), **BAD[case]}
    with pytest.raises(ValueError):
        wg.wg_decode_step(FakeContext(), a["gid"], a["sid"], a["logits"], a["bitmask"],
                          a["token_out"], a["status"])
    with pytest.raises(ValueError):
        wg.StepGraph(FakeContext(), a["gid"], a["sid"], a["logits"], a["bitmask"], a["token_out"],
                     a["status"])


def test_step_plan_refuses(no_library):
    a = good()
    with pytest.raises(ValueError):
        wg.StepPlan(FakeContext(), FakeTensor([B + 1]), a["sid"], a["bitmask"], a["token_out"])
    with pytest.raises(ValueError):
        wg.StepPlan(FakeContext(), a["gid"], a["sid"], a["bitmask"], a["token_out"],
                    FakeTensor([B - 1]))
    with pytest.raises(ValueError):
        wg.StepPlan(FakeContext(), a["gid"], a["sid"], FakeTensor([B, W - 1]), a["token_out"])


def test_build_masks_advance_and_lookup_refuse(no_library):
    a = good()
    with pytest.raises(ValueError):
        wg.wg_build_masks(FakeContext(), FakeTensor([B - 1]), a["sid"], a["bitmask"])
    with pytest.raises(ValueError):
        wg.wg_build_masks(FakeContext(), a["gid"], a["sid"], FakeTensor([B, W - 1]))
    with pytest.raises(ValueError):
        wg.wg_advance(FakeContext(), a["gid"], FakeTensor([B - 1]), a["token_out"])
    with pytest.raises(ValueError):
        wg.wg_advance(FakeContext(), a["gid"], a["sid"], a["token_out"], FakeTensor([B - 1]))
    with pytest.raises(ValueError):
        wg.wg_mask_cache_lookup(FakeContext(), a["gid"], a["sid"], FakeTensor([B - 1]))
    with pytest.raises(ValueError):
        wg.wg_advance_keys(FakeContext(), a["gid"], a["sid"], FakeTensor([B - 1], torch.int64),
                           a["token_out"])
    with pytest.raises(TypeError):
        wg.wg_advance(FakeContext(), a["gid"], a["sid"], FakeTensor([B], torch.int64))


def test_apply_mask_refuses(no_library):
    a = good()
    ws = FakeTensor([8 * B], torch.uint8)
    with pytest.raises(ValueError):                 # mask rows shorter than ceil(V / 32) words
        wg.wg_apply_mask(a["logits"], FakeTensor([B, W - 1]), V)
    with pytest.raises(ValueError):                 # fewer mask rows than logits rows
        wg.wg_apply_mask(a["logits"], FakeTensor([B - 1, W]), V)
    with pytest.raises(ValueError):                 # V beyond the row length
        wg.wg_apply_mask(a["logits"], a["bitmask"], V + 1)
    with pytest.raises(ValueError):                 # workspace too small for the argmax
        wg.wg_apply_mask(a["logits"], a["bitmask"], V, a["token_out"], FakeTensor([8 * B - 1], torch.uint8))
    with pytest.raises(ValueError):                 # argmax without a workspace
        wg.wg_apply_mask(a["logits"], a["bitmask"], V, a["token_out"], None)
    with pytest.raises(ValueError):                 # token array shorter than the batch
        wg.wg_apply_mask(a["logits"], a["bitmask"], V, FakeTensor([B - 1]), ws)
    with pytest.raises(ValueError):                 # mask on another device than the logits
        wg.wg_apply_mask(a["logits"], FakeTensor([B, W], device=1), V)
    with pytest.raises(ValueError):
        wg.wg_apply_mask_noalloc(a["logits"], a["bitmask"], V, FakeTensor([B - 1]))


def test_host_step_refuses(no_library):
    a = good()
    host = torch.zeros((B, V))
    tok_host = torch.zeros(B, dtype=torch.int32)
    call = lambda **kw: wg.wg_decode_step_host(      # noqa: E731
        FakeContext(), a["gid"], a["sid"], kw.get("host", host), a["logits"], a["bitmask"],
        kw.get("tok", a["token_out"]), kw.get("tok_host", tok_host), a["status"])
    with pytest.raises(ValueError):
        call(host=torch.zeros((B - 1, V)))
    with pytest.raises(ValueError):
        call(host=torch.zeros((B, V), dtype=torch.bfloat16))
    with pytest.raises(ValueError):
        call(tok_host=torch.zeros(B - 1, dtype=torch.int32))
    with pytest.raises(ValueError):
        call(tok=FakeTensor([B - 1]))


def test_mask_only_step_takes_no_status_and_no_restart_flag(no_library):
    a = good()
    with pytest.raises(ValueError):
        wg.wg_decode_step(FakeContext(), a["gid"], a["sid"], a["logits"], a["bitmask"], None, a["status"])
    with pytest.raises(ValueError):
        wg.wg_decode_step(FakeContext(), a["gid"], a["sid"], a["logits"], a["bitmask"], None, None,
                          wg.WG_USE_CACHE | wg.WG_RESTART_ON_DONE)
