"""Shared test helpers (input plumbing only; no method arithmetic)."""
import os

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(ROOT, "tests", "golden")


def read_records(name):
    """Parse a golden file of blank-line separated 'key: value' records."""
    records, cur = [], {}
    with open(os.path.join(GOLDEN, name), encoding="utf-8") as fh:
        for line in fh:
            line = line.rstrip("\n")
            if line.startswith("#"):
                continue
            if not line.strip():
                if cur:
                    records.append(cur)
                    cur = {}
                continue
            key, _, value = line.partition(": ")
            cur[key] = value
    if cur:
        records.append(cur)
    return records


def read_regexes(name="paper_regexes.txt"):
    out = {}
    with open(os.path.join(GOLDEN, name), encoding="utf-8") as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, _, value = line.rstrip("\n").partition("\t")
            out[key] = value
    return out


def split_tokens(s):
    return [t.encode("latin-1") for t in s.split(" | ")]


def column_classes(trans):
    """One representative byte per group of bytes the DFA never tells apart."""
    _, first = np.unique(np.asarray(trans).T, axis=0, return_index=True)
    return sorted(int(b) for b in first)
