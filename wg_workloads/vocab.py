"""Seeded synthetic vocabularies in CSR form.

Token ids 0..255 are the single bytes (token i = byte i) except ``eos_id``
(2), which is the end-of-sequence token and has no byte string.  Every other
token is a unique byte string whose length is Geometric(p = 0.25) clipped to
1..16 and whose bytes are drawn per position from five classes: 55 % ASCII
letters, 10 % digits, 15 % whitespace, 15 % structural characters, 5 % other
UTF-8.  A draw that repeats an earlier token (the single bytes included) is
redrawn as a whole.
"""
from __future__ import annotations

from dataclasses import dataclass
from functools import lru_cache

import numpy as np

EOS_ID = 2
MAX_LEN = 16

LETTERS = np.frombuffer(b"abcdefghijklmnopqrstuvwxyzABCDEFGHIJKLMNOPQRSTUVWXYZ", dtype=np.uint8)
DIGIT_BYTES = np.frombuffer(b"0123456789", dtype=np.uint8)
WHITESPACE = np.frombuffer(b" \n\t\r", dtype=np.uint8)
STRUCTURAL = np.frombuffer(b"<>/\"{}:,=[]", dtype=np.uint8)
# printable ASCII outside the four classes above: the one-byte stand-in for "other"
# when a two-byte UTF-8 sequence no longer fits
OTHER_ASCII = np.frombuffer(b"!#$%&'()*+-.;?@\\^_`|~", dtype=np.uint8)
CLASS_CDF = np.cumsum([0.55, 0.10, 0.15, 0.15, 0.05])


@dataclass(frozen=True)
class Vocab:
    offsets: np.ndarray  # uint32 [V + 1]
    data: np.ndarray     # uint8 [offsets[-1]]
    eos_id: int

    @property
    def size(self) -> int:
        return int(self.offsets.shape[0] - 1)

    def token(self, t: int) -> bytes:
        return self.data[self.offsets[t]:self.offsets[t + 1]].tobytes()

    def tokens(self):
        d = self.data.tobytes()
        o = self.offsets
        return [d[o[t]:o[t + 1]] for t in range(self.size)]

    def lengths(self) -> np.ndarray:
        return np.diff(self.offsets.astype(np.int64)).astype(np.int32)


def vocab_from_tokens(tokens, eos_id: int = EOS_ID) -> Vocab:
    """CSR vocabulary from an explicit list of byte strings (tests, tiny cases)."""
    lens = np.array([len(t) for t in tokens], dtype=np.int64)
    offsets = np.zeros(len(tokens) + 1, dtype=np.uint32)
    offsets[1:] = np.cumsum(lens)
    data = np.frombuffer(b"".join(bytes(t) for t in tokens), dtype=np.uint8).copy()
    return Vocab(offsets=offsets, data=data, eos_id=int(eos_id))


def _draw_batch(rng: np.random.Generator, n_tok: int):
    """``n_tok`` candidate tokens as a padded byte matrix [n_tok, 16] and lengths."""
    n = np.minimum(MAX_LEN, rng.geometric(0.25, size=n_tok)).astype(np.int64)
    cls = np.searchsorted(CLASS_CDF, rng.random((n_tok, MAX_LEN)), side="right")
    pick = rng.integers(0, 1 << 30, size=(n_tok, MAX_LEN), dtype=np.int64)
    pick2 = rng.integers(0, 64, size=(n_tok, MAX_LEN), dtype=np.int64)
    out = np.zeros((n_tok, MAX_LEN + 1), dtype=np.uint8)
    pos = np.zeros(n_tok, dtype=np.int64)
    rows = np.arange(n_tok)
    for j in range(MAX_LEN):
        active = pos < n
        if not active.any():
            break
        c = cls[:, j]
        r = pick[:, j]
        # "other": a valid two-byte UTF-8 sequence (lead 0xC2..0xDF, continuation
        # 0x80..0xBF) while two bytes of room remain, else one printable ASCII byte
        two = active & (c == 4) & (n - pos >= 2)
        b = np.select(
            [c == 0, c == 1, c == 2, c == 3, two],
            [LETTERS[r % LETTERS.size], DIGIT_BYTES[r % DIGIT_BYTES.size],
             WHITESPACE[r % WHITESPACE.size], STRUCTURAL[r % STRUCTURAL.size],
             (0xC2 + r % 30).astype(np.uint8)],
            default=OTHER_ASCII[r % OTHER_ASCII.size]).astype(np.uint8)
        wpos = np.where(active, pos, MAX_LEN)  # inactive rows write into the spare column
        out[rows, wpos] = b
        pos = pos + active
        wpos2 = np.where(two, pos, MAX_LEN)
        out[rows, wpos2] = (0x80 + pick2[:, j]).astype(np.uint8)
        pos = pos + two
    return out[:, :MAX_LEN], n


@lru_cache(maxsize=8)
def make_vocab(V: int, seed: int, eos_id: int = EOS_ID) -> Vocab:
    if V < 256:
        raise ValueError("the generated vocabularies start with the 256 single bytes")
    rng = np.random.Generator(np.random.Philox(key=[seed, 0x766F636162]))
    tokens = [bytes([i]) for i in range(256)]
    tokens[eos_id] = b""
    seen = set(tokens)
    seen.add(bytes([eos_id]))  # byte 0x02 has no token of its own
    while len(tokens) < V:
        mat, n = _draw_batch(rng, max(1024, int(1.3 * (V - len(tokens)))))
        flat = mat.tobytes()
        for i in range(mat.shape[0]):
            t = flat[i * MAX_LEN:i * MAX_LEN + int(n[i])]
            if t in seen:
                continue  # a repeated draw is dropped whole and drawn again
            seen.add(t)
            tokens.append(t)
            if len(tokens) == V:
                break
    return vocab_from_tokens(tokens, eos_id)


def has_structural_byte(vocab: Vocab, chars: bytes = b"") -> np.ndarray:
    """bool [V]: the token contains one of ``chars`` (default: the structural characters).

    Input shaping only: the benchmark and the tests add a constant to the logits of these tokens
    so that greedy decoding leaves free-text slots."""
    is_struct = np.zeros(256, dtype=bool)
    is_struct[np.frombuffer(chars, dtype=np.uint8) if chars else STRUCTURAL] = True
    hit = is_struct[vocab.data]
    csum = np.zeros(vocab.data.shape[0] + 1, dtype=np.int64)
    csum[1:] = np.cumsum(hit)
    o = vocab.offsets.astype(np.int64)
    return (csum[o[1:]] - csum[o[:-1]]) > 0
