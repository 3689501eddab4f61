"""The seeded input generators are reproducible and have the stated shapes."""
import hashlib

import numpy as np

from synth import (gumbel_noise, make_vocab_api, make_vocab_geometric, normal_logits,
                   random_range_dfa, schema40_regex)
from synth.configs import CONFIGS, config_dfas, row_table_for
from synth.models import draft_logits, prefix_key, target_logits


def digest(*arrays):
    h = hashlib.sha256()
    for a in arrays:
        h.update(np.ascontiguousarray(a).tobytes())
    return h.hexdigest()


def test_vocabularies():
    vb, vo = make_vocab_api(0)
    assert vo.size - 1 == 1024 and (vb[:256] == np.arange(256)).all()
    lens = vo[1:] - vo[:-1]
    assert (lens[:256] == 1).all() and lens[256:].min() >= 2 and lens[256:].max() <= 6
    assert set(vb[256:].tolist()) <= set(b'abcdefghijklmnopqrstuvwxyz0123456789_(),=" ')
    vb2, vo2 = make_vocab_geometric(32000, 0)
    lens = vo2[1:] - vo2[:-1]
    assert vo2.size - 1 == 32000 and lens.max() <= 16 and lens.min() >= 1
    assert abs(float(lens[256:].mean()) - 3.3) < 0.1                # Geometric(0.3) capped at 16
    chars = vb2[256:]
    assert abs(float(((chars >= 97) & (chars <= 122)).mean()) - 0.60) < 0.01
    assert abs(float((chars == 32).mean()) - 0.15) < 0.01
    assert digest(*make_vocab_geometric(32000, 0)) == digest(vb2, vo2)
    assert digest(*make_vocab_geometric(32000, 1)) != digest(vb2, vo2)


def test_random_dfa_recipe():
    trans, accept, start = random_range_dfa(500, seed=2)
    assert trans.shape == (500, 256) and start == 0 and trans.max() < 500 and trans.min() == -1
    for q in range(500):
        live = trans[q] >= 0
        ranges = int((live[1:] & ~live[:-1]).sum() + live[0])       # maximal runs of live bytes
        assert 1 <= ranges <= 16                                    # adjacent ranges may merge into one run
    assert 0.1 < accept.mean() < 0.3
    assert digest(*random_range_dfa(500, seed=2)[:2]) == digest(trans, accept)


def test_logits_rows_are_independent_of_the_batch():
    a = normal_logits(100, 3, range(8), 1000)
    b = normal_logits(100, 3, [5], 1000)
    assert np.array_equal(a[5], b[0])
    assert not np.array_equal(a[4], a[5])
    g = gumbel_noise(1, 0, [2, 7], 1000)
    assert np.isfinite(g).all() and np.array_equal(g[1], gumbel_noise(1, 0, [7], 1000)[0])
    assert abs(float(normal_logits(7, 0, range(64), 4000, sigma=2.0).std()) - 2.0) < 0.02
    padded = normal_logits(100, 3, [5], 1000, ld=1008)
    assert padded.shape == (1, 1008) and np.array_equal(padded[0, :1000], b[0]) and not padded[0, 1000:].any()


def test_workloads_and_models():
    assert [CONFIGS[n].vocab_size for n in CONFIGS] == [1024, 32000, 128256, 256000, 256000]
    assert [CONFIGS[n].batch for n in CONFIGS] == [4, 64, 256, 512, 1024]
    assert schema40_regex(0) == schema40_regex(0) and schema40_regex(0).count('"k') == 40
    assert [d[0].shape[0] for d in (config_dfas("api_1k")[0], config_dfas("json_32k")[0])] == [11, 56]
    rt = row_table_for(CONFIGS["random10k_256k"])
    assert rt.shape == (1024,) and (np.bincount(rt) == 128).all()
    assert prefix_key([1, 2]) != prefix_key([2, 1]) and prefix_key([]) == prefix_key(())
    t = target_logits(3, 0, [4, 5], 500)
    assert np.array_equal(t, target_logits(3, 0, [4, 5], 500))
    d = draft_logits(3, 0, [4, 5], 500)
    assert not np.array_equal(t, d) and np.corrcoef(t, d)[0, 1] > 0.7


def test_pushdown_inputs_are_seeded_and_well_formed():
    from synth import json_grammar_pda, json_pda, make_vocab_json, random_pda
    vb, vo = make_vocab_json(5000, seed=3)
    vb2, vo2 = make_vocab_json(5000, seed=3)
    assert np.array_equal(vb, vb2) and np.array_equal(vo, vo2)
    toks = [bytes(vb[vo[v]:vo[v + 1]]) for v in range(vo.size - 1)]
    assert toks[:256] == [bytes([c]) for c in range(256)]
    assert b"]]" in toks and b'{"' in toks and b"" in toks and len(toks) == 5000
    for P in (json_pda(), json_grammar_pda(), random_pda(5), random_pda(5)):
        n = P.n_edges
        assert P.pop_off.size == n + 1 and P.push_off.size == n + 1
        assert P.pop_off[-1] == P.pops.size and P.push_off[-1] == P.pushes.size
        assert P.src.min() >= 0 and P.src.max() < P.n_states and P.tgt.max() < P.n_states
        assert (P.pops < P.n_symbols).all() and (P.pushes < P.n_symbols).all()
        assert np.diff(P.pop_off).max() <= 1 and np.diff(P.push_off).max() <= 3
    a, b = random_pda(5), random_pda(5)
    assert np.array_equal(a.src, b.src) and np.array_equal(a.pushes, b.pushes)
