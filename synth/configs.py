"""The five synthetic workloads (constraint, vocabulary, batch, decoding recipe).

Each stands in for a real deployment shape: an LM vocabulary of a common size
(1k toy, 32k, 128k, 256k as in the paper's Section 5.1 measurements) against a
regex-derived or random byte DFA, decoded for a batch of rows that all start
at the DFA's start state.
"""

from __future__ import annotations

from dataclasses import dataclass, field
from functools import lru_cache

import numpy as np

from . import constraints, vocab
from .regex_frontend import regex_to_dfa


@dataclass(frozen=True)
class Workload:
    name: str
    vocab_size: int
    batch: int
    steps: int
    dtype: str            # "f32" or "bf16"
    sigma: float          # logits ~ N(0, sigma^2)
    gumbel: bool          # Gumbel-max with supplied noise (seed 1) instead of greedy
    regex: str | None = None
    n_dfas: int = 1       # > 1: mixed-constraint batch, equal row blocks per DFA
    dfa_states: int = 0   # random-DFA workloads only
    dfa_seed0: int = 2
    vocab_kind: str = "geometric"
    logits_seed: int = 100
    noise_seed: int = 1
    extra: dict = field(default_factory=dict)


CONFIGS = {
    "api_1k": Workload("api_1k", 1024, 4, 32, "f32", 1.0, False,
                       regex=constraints.API_CALL_REGEX, vocab_kind="api"),
    "json_32k": Workload("json_32k", 32000, 64, 256, "bf16", 2.0, False,
                         regex=constraints.FLAT_JSON_REGEX),
    "schema40_128k": Workload("schema40_128k", 128256, 256, 512, "f32", 1.0, True,
                              regex="<schema40>"),
    "string_256k": Workload("string_256k", 256000, 512, 128, "f32", 1.0, False,
                            regex=constraints.STRING_LITERAL_REGEX),
    "random10k_256k": Workload("random10k_256k", 256000, 1024, 64, "f32", 1.0, False,
                               n_dfas=8, dfa_states=10000, dfa_seed0=2),
}


def get_config(name: str) -> Workload:
    return CONFIGS[name]


@lru_cache(maxsize=None)
def config_vocab(name: str):
    w = CONFIGS[name]
    if w.vocab_kind == "api":
        return vocab.make_vocab_api(seed=0)
    return vocab.make_vocab_geometric(w.vocab_size, seed=0)


@lru_cache(maxsize=None)
def config_dfas(name: str, scale_states: int | None = None):
    """List of (trans, accept, start) for the workload (one entry unless mixed)."""
    w = CONFIGS[name]
    if w.regex is not None:
        pattern = constraints.schema40_regex(seed=0) if w.regex == "<schema40>" else w.regex
        return [regex_to_dfa(pattern)]
    n = w.dfa_states if scale_states is None else scale_states
    return [constraints.random_range_dfa(n, seed=w.dfa_seed0 + g) for g in range(w.n_dfas)]


def row_table_for(w: Workload, batch: int | None = None) -> np.ndarray | None:
    """Per-row table index for mixed-constraint batches: equal contiguous blocks."""
    if w.n_dfas <= 1:
        return None
    b = w.batch if batch is None else batch
    per = max(b // w.n_dfas, 1)
    return np.minimum(np.arange(b) // per, w.n_dfas - 1).astype(np.int32)
