"""Constraint inputs: the regexes of the regex-derived workloads and the random
byte-range DFAs of the table-build scaling workload.

A byte-level DFA is the triple the C ABI loads: ``trans`` int32 ``[S][256]``
(target state, or -1 where the state has no edge on that byte), ``accept``
uint8 ``[S]`` and a start state.
"""

from __future__ import annotations

import numpy as np

# API call such as foo(x="bar", n=12) (the paper's Section 1 example shape).
API_CALL_REGEX = (
    r'[a-z_][a-z0-9_]*\(([a-z]+=("[a-z ]*"|[0-9]+)(, [a-z]+=("[a-z ]*"|[0-9]+))*)?\)'
)

_STR = r'"[^"\\]*"'
_INT = r"-?[0-9]{1,3}"

# Flat JSON object with keys name / age / tags in fixed order; one optional
# space after ':' and ','; tags holds 0..5 strings.
FLAT_JSON_REGEX = (
    r'\{"name": ?' + _STR + r', ?"age": ?' + _INT + r', ?"tags": ?\[('
    + _STR + r"(, ?" + _STR + r"){0,4})?\]\}"
)

# A double-quoted string literal of at most 4096 items, an item being any byte
# other than quote / backslash, or a backslash followed by any byte.
STRING_LITERAL_REGEX = r'"([^"\\]|\\.){0,4096}"'


# Small constraints of the kinds the paper times in its Table 1 (a multiple-choice answer, an
# ISO date-time, an IPv4 address), written here from their usual definitions.
SMALL_CONSTRAINTS = {
    "multiple_choice": r"(A|B|C|D)",
    "iso_date_time": r"[0-9]{4}-[0-9]{2}-[0-9]{2}T[0-9]{2}:[0-9]{2}:[0-9]{2}(Z|[+-][0-9]{2}:[0-9]{2})",
    "ipv4_address": r"((25[0-5]|2[0-4][0-9]|1?[0-9]?[0-9])\.){3}(25[0-5]|2[0-4][0-9]|1?[0-9]?[0-9])",
}


def schema40_regex(seed: int = 0, n_keys: int = 40) -> str:
    """JSON object with ``n_keys`` required keys k00.. in fixed order; value
    types cycle string / integer / true|false / enum of 8 seeded random
    lowercase literals of 3..10 letters; one optional space after ':' and ','."""
    rng = np.random.Generator(np.random.PCG64(seed))
    parts = []
    for k in range(n_keys):
        kind = k % 4
        if kind == 0:
            val = _STR
        elif kind == 1:
            val = _INT
        elif kind == 2:
            val = "(true|false)"
        else:
            lits = []
            while len(lits) < 8:
                n = int(rng.integers(3, 11))
                s = "".join(chr(0x61 + int(c)) for c in rng.integers(0, 26, size=n))
                if s not in lits:
                    lits.append(s)
            val = '"(' + "|".join(lits) + ')"'
        parts.append('"k%02d": ?%s' % (k, val))
    return r"\{" + ", ?".join(parts) + r"\}"


def random_range_dfa(n_states: int = 10000, seed: int = 2, accept_prob: float = 0.2):
    """Random byte DFA: each state has k ~ U{4..16} disjoint outgoing byte
    ranges (2k distinct sorted cut points in 0..256, ranges [c0,c1), [c2,c3),
    ...), each range going to one uniform random target; all other bytes have
    no edge; a state accepts with probability ``accept_prob``; start state 0."""
    rng = np.random.Generator(np.random.PCG64(seed))
    trans = np.full((n_states, 256), -1, dtype=np.int32)
    ks = rng.integers(4, 17, size=n_states)
    for q in range(n_states):
        k = int(ks[q])
        cuts = np.sort(rng.choice(257, size=2 * k, replace=False))
        targets = rng.integers(0, n_states, size=k)
        for i in range(k):
            trans[q, cuts[2 * i]:cuts[2 * i + 1]] = targets[i]
    accept = (rng.random(n_states) < accept_prob).astype(np.uint8)
    return trans, accept, 0
