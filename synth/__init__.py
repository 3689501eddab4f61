"""Seeded synthetic inputs for regular-language constrained decoding.

Everything here produces *inputs* (vocabularies, byte-level DFAs, logits,
Gumbel noise) for the token-table builder and the constrained step.  None of
the method's own arithmetic (walking token bytes through a DFA, masking,
selecting, advancing) lives in this package, so both the CUDA library and the
CPU oracle can be fed from it without sharing any code with each other.
"""

from .vocab import (make_vocab_api, make_vocab_geometric, make_vocab_json,  # noqa: F401
                    vocab_from_strings)
from .constraints import (  # noqa: F401
    API_CALL_REGEX,
    FLAT_JSON_REGEX,
    STRING_LITERAL_REGEX,
    schema40_regex,
    random_range_dfa,
)
from .logits import normal_logits, gumbel_noise, f32_to_bf16_bits, bf16_bits_to_f32  # noqa: F401
from .regex_frontend import regex_to_dfa  # noqa: F401
from .configs import CONFIGS, get_config  # noqa: F401
from .pda import (Pda, PdaBuilder, anbn_pda, dyck_pda, json_pda, random_pda,  # noqa: F401
                  stackless_pda)
from .grammar import GrammarError, anbn_grammar_pda, grammar_to_pda, json_grammar_pda  # noqa: F401
