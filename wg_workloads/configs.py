"""The five workload configurations: sizes, dtypes and how each batch row picks a grammar."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List

from . import grammars
from .optree import Op


@dataclass(frozen=True)
class Workload:
    name: str
    V: int
    batch: int
    steps: int
    dtype: str            # "fp32" or "bf16"
    vocab_seed: int
    use_cache: bool
    prewarm: bool
    n_grammars: int
    description: str

    @property
    def steer_bytes(self) -> bytes:
        """Characters whose tokens get the steering bonus (empty = all structural ones).

        The snippet workload only favours '<': a row then leaves a free-text slot on its next
        step, so leaders keep meeting new states and the cache hit rate comes from the
        followers (about one half), as the workload asks."""
        return b"<" if self.name == "dynamic_snippets" else b""

    def grammar(self, g: int) -> Op:
        return _GRAMMARS[self.name](g)

    def grammar_of_row(self, row: int) -> int:
        if self.name == "dynamic_snippets":
            return row // 2       # leader / follower pairs share one instantiation
        return row % self.n_grammars

    def row_delay(self, row: int) -> int:
        """Steps a row waits before its request starts (followers trail leaders by one)."""
        if self.name == "dynamic_snippets":
            return row % 2
        return 0


_GRAMMARS: dict[str, Callable[[int], Op]] = {
    "html_tiny": lambda g: grammars.html_template(),
    "json_lookup": lambda g: grammars.json_reference_lookup(),
    "cold_templates": lambda g: grammars.random_template(seed=g),
    "json_warm": lambda g: grammars.json_reference_lookup(),
    "html_warm_free_text": lambda g: grammars.html_template(),
    "dynamic_snippets": lambda g: grammars.dynamic_snippet_template(seed=g),
}

WORKLOADS: List[Workload] = [
    Workload("html_tiny", 32000, 1, 256, "fp32", 1, True, False, 1,
             "tiny HTML-template decode, batch 1"),
    Workload("json_lookup", 128256, 32, 512, "bf16", 2, True, False, 1,
             "JSON reference-lookup, batch 32"),
    Workload("cold_templates", 151936, 256, 256, "bf16", 3, False, False, 8,
             "cold-cache build stress: 8 random templates, cache disabled"),
    Workload("json_warm", 128256, 1024, 1024, "bf16", 4, True, True, 1,
             "cache-warm steady state: prewarmed cache, gather + apply"),
    Workload("dynamic_snippets", 256000, 128, 512, "fp32", 5, True, False, 64,
             "large dynamic-snippet grammar: 64 instantiations shared by row pairs"),
]

# Not one of the five configurations: the cache-warm steady state of workload 4 with every row
# dwelling in a free-text slot (the HTML template on unsteered logits walks through its first tag
# and then stays in the slot), so that nearly every token is allowed and the apply pass reads
# every logit instead of overwriting it.  A diagnostic for the apply kernel's other extreme.
EXTRA_WORKLOADS: List[Workload] = [
    Workload("html_warm_free_text", 128256, 1024, 256, "bf16", 4, True, True, 1,
             "cache-warm steady state with rows in free-text slots (mostly-allowed masks)"),
]

BY_NAME = {w.name: w for w in WORKLOADS + EXTRA_WORKLOADS}
