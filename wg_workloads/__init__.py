"""Seeded synthetic inputs (vocabularies, operator trees, logits) for tests and benchmarks.

This package describes inputs only.  It contains none of the masking, matching or table
arithmetic: the CPU checker and the CUDA library each read these arrays with code of their own.
"""
from .optree import (ALL_BYTES, DIGITS, EOS, Cond, DoWhile, FlatTree, Hole, IfElse, Op, Sequence,
                     Switch, SymSet, Wait, WaitUntil, Write, WriteTokens, enum_trie, flatten,
                     substitute)
from .vocab import EOS_ID, Vocab, has_structural_byte, make_vocab, vocab_from_tokens
from .logits import bf16_bits_to_f32, f32_to_bf16_bits, make_logits
from .configs import BY_NAME, WORKLOADS, Workload
from . import grammars
