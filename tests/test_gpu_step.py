"""GPU parity: the fused constrained step vs the CPU oracle, bit exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_08103_b200 import cstr
from paper_2407_08103_b200.decode import ConstrainedDecoder
from synth import (f32_to_bf16_bits, gumbel_noise, normal_logits, random_range_dfa,
                   vocab_from_strings)
from synth.configs import CONFIGS, config_dfas, config_vocab, row_table_for
from synth.regex_frontend import regex_to_dfa

from gpu_common import DEV, bits_equal, from_dev_logits, gpu_tables, run_step_both, to_dev_logits
from test_gpu_table import dense_random_dfa, random_vocab

pytestmark = pytest.mark.gpu


def rand_logits(rng, B, V, ld, dtype):
    x = np.zeros((B, ld), dtype=np.float32)
    x[:, :V] = rng.standard_normal((B, V)).astype(np.float32)
    x[:, V:] = 50.0                         # padding larger than any logit: must be ignored
    return x if dtype == "f32" else f32_to_bf16_bits(x)


@pytest.mark.parametrize("seed", range(16))
def test_random_small(seed):
    rng = np.random.default_rng(100 + seed)
    S = int(rng.choice([1, 3, 40, 300]))
    V = int(rng.choice([1, 7, 32, 33, 1000, 1024, 1027, 4096, 9001, 20000]))
    B = int(rng.choice([1, 2, 5, 33]))
    dtype = "bf16" if seed % 2 else "f32"
    align = 8 if dtype == "bf16" else 4
    ld = V if seed % 4 < 2 else (V + align - 1) // align * align + align   # unaligned and padded strides
    dfa = dense_random_dfa(rng, S, live=float(rng.choice([0.05, 0.6, 1.0])))
    vb, vo = random_vocab(rng, V, max_len=6)
    tables = gpu_tables([dfa], vb, vo)
    logits = rand_logits(rng, B, V, ld, dtype)
    states = rng.integers(-1, S, size=B).astype(np.int32)
    noise = None
    if seed % 3 == 0:
        noise = np.zeros((B, ld), dtype=np.float32)
        noise[:, :V] = -np.log(-np.log(rng.random((B, V)))).astype(np.float32)
    run_step_both([dfa], tables, vb, vo, logits, states, noise=noise, in_place=(seed % 5 == 0))


def test_ties_signed_zero_nan_inf_across_chunks():
    # Several chunks per row (V spans many tiles); the tie / NaN / inf rules
    # must hold across CTA boundaries, not only inside one thread.
    V, B = 70000, 8
    dfa = (np.zeros((1, 256), dtype=np.int32), np.ones(1, dtype=np.uint8), 0)   # everything allowed
    toks = [bytes([65 + i % 26]) for i in range(V)]
    vb, vo = vocab_from_strings(toks)
    tables = gpu_tables([dfa], vb, vo)
    x = np.full((B, V), -3.0, dtype=np.float32)
    x[0, [100, 40000, 69999]] = 2.5                  # equal maxima in three chunks: lowest id
    x[1, 50000] = -0.0; x[1, 60000] = 0.0; x[1, :] = np.where(x[1] == -3.0, -1.0, x[1])   # -0 == +0: lowest id
    x[2, 60000] = -0.0; x[2, 50000] = 0.0; x[2, :] = np.where(x[2] == -3.0, -1.0, x[2])
    x[3, :] = np.nan; x[3, 65000] = -np.inf          # a -inf beats NaNs
    x[4, :] = np.nan                                 # nothing selectable
    x[5, 123] = np.inf; x[5, 69000] = np.inf
    x[6, :] = -np.inf                                # all -inf: token 0
    x[7, 33333] = np.float32(1e-45)                  # denormal vs negatives
    ref = run_step_both([dfa], tables, vb, vo, x, np.zeros(B, dtype=np.int32))
    assert ref["tokens"].tolist() == [100, 50000, 50000, 65000, -1, 123, 0, 33333]
    # the same with noise whose sum creates ties and NaN (inf + -inf)
    noise = np.zeros((B, V), dtype=np.float32)
    noise[0, 100] = -1.0
    noise[5, 123] = -np.inf
    ref = run_step_both([dfa], tables, vb, vo, x, np.zeros(B, dtype=np.int32), noise=noise)
    assert ref["tokens"][0] == 40000 and ref["tokens"][5] == 69000


def test_inactive_bad_and_empty_rows():
    dfa = regex_to_dfa("(a|b)*c")
    toks = [b"a", b"b", b"c", b"ab", b"zz", b"bc", b"ca"] + [b"q%d" % i for i in range(3000)]
    vb, vo = vocab_from_strings(toks)
    tables = gpu_tables([dfa], vb, vo)
    V = len(toks)
    S = dfa[0].shape[0]
    acc_state = int(np.nonzero(dfa[1])[0][0])
    states = np.array([-1, S, -7, 2 ** 30, dfa[2], acc_state], dtype=np.int32)
    rng = np.random.default_rng(0)
    for dtype in ("f32", "bf16"):
        logits = rand_logits(rng, 6, V, (V + 7) // 8 * 8, dtype)
        ref = run_step_both([dfa], tables, vb, vo, logits, states)
        assert ref["bad_state_rows"] == 3 and ref["empty_mask_rows"] == 1


def test_eos_token():
    dfa = regex_to_dfa("ab?")
    toks = [b"a", b"b", b"<eos>", b"ab"]
    vb, vo = vocab_from_strings(toks)
    tables = gpu_tables([dfa], vb, vo, eos_id=2)
    logits = np.array([[0.0, 0.0, 5.0, 1.0]] * 3, dtype=np.float32)
    states = np.arange(3, dtype=np.int32) % dfa[0].shape[0]
    run_step_both([dfa], tables, vb, vo, logits, states, eos_id=2)


def test_mixed_tables_and_bad_table_index():
    rng = np.random.default_rng(4)
    V = 5000
    vb, vo = random_vocab(rng, V, max_len=5)
    dfas = [dense_random_dfa(rng, S) for S in (5, 70, 300)]
    tables = gpu_tables(dfas, vb, vo)
    B = 24
    row_table = rng.integers(0, 3, size=B).astype(np.int32)
    row_table[3] = 3        # out of range
    row_table[9] = -1
    states = np.array([rng.integers(0, dfas[min(max(t, 0), 2)][0].shape[0]) for t in row_table],
                      dtype=np.int32)
    logits = rand_logits(rng, B, V, V, "f32")
    ref = run_step_both(dfas, tables, vb, vo, logits, states, row_table=row_table)
    assert ref["tokens"][3] == -1 and ref["tokens"][9] == -1 and ref["bad_state_rows"] == 2


def test_wide_table_entries():
    # more than 32,766 states: 32-bit table entries, decoded by the step's last-arriving CTA
    rng = np.random.default_rng(12)
    dfa = random_range_dfa(33000, seed=9)
    vb, vo = random_vocab(rng, 300, max_len=3)
    tables = gpu_tables([dfa], vb, vo)
    V = vo.size - 1
    states = np.array([0, 1, 32766, 32767, 32768, 32999, 33000, -1], dtype=np.int32)
    for dtype in ("f32", "bf16"):
        logits = rand_logits(rng, 8, V, (V + 7) // 8 * 8, dtype)
        ref = run_step_both([dfa], tables, vb, vo, logits, states)
        assert ref["bad_state_rows"] == 1 and (ref["tokens"][:6] >= 0).any()


def test_error_codes_on_device_arguments():
    dfa = regex_to_dfa("a*")
    vb, vo = vocab_from_strings([b"a", b"b", b"aa"])
    vb2, vo2 = vocab_from_strings([b"a", b"b"])
    (t3,) = gpu_tables([dfa], vb, vo)
    (t2,) = gpu_tables([dfa], vb2, vo2)
    ws = cstr.cstr_workspace_create(2)
    logits = torch.zeros(2, 3, device=DEV)
    st = torch.zeros(2, dtype=torch.int32, device=DEV)
    tok = torch.zeros(2, dtype=torch.int32, device=DEV)
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_step([t3, t2], logits, st, tok, torch.empty_like(logits), ws)
    assert e.value.code == -6
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_step([t3], logits, st, tok, torch.empty_like(logits), ws, vocab_ld=2)
    assert e.value.code == -6
    big = torch.zeros(3, 3, device=DEV)
    st3 = torch.zeros(3, dtype=torch.int32, device=DEV)
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_step([t3], big, st3, st3.clone(), torch.empty_like(big), ws)
    assert e.value.code == -6
    unbuilt = cstr.cstr_table_create(t3.vocab, 4)
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_step([unbuilt], logits, st, tok, torch.empty_like(logits), ws)
    assert e.value.code == -2
    with pytest.raises(cstr.CstrError):
        cstr.cstr_table_download(t3, 0, 99)


def decode_and_check(name, steps=None, pool=2, batch=None):
    """Decode a workload on the GPU for `steps` steps (default: the workload's own
    length), logits cycling through a pool of `pool` seeded tensors, and replay every
    step on the oracle for ALL rows: tokens, states, accept flags and every masked
    logit are compared bit for bit at every step.  The oracle's own states feed its
    next step, so a row that finishes must stay finished on both sides."""
    w = CONFIGS[name]
    B = w.batch if batch is None else batch
    steps = w.steps if steps is None else steps
    dfas = config_dfas(name)
    vb, vo = config_vocab(name)
    V = vo.size - 1
    tables = gpu_tables(dfas, vb, vo)
    row_table = row_table_for(w, B)
    dec = ConstrainedDecoder(tables, B, row_table=row_table)
    pools, noises = [], []
    for k in range(pool):
        pools.append(normal_logits(w.logits_seed, k, range(B), V, sigma=w.sigma, dtype=w.dtype))
        noises.append(gumbel_noise(w.noise_seed, k, range(B), V) if w.gumbel else None)
    d_pool = [to_dev_logits(p) for p in pools]
    d_noise = [None if n is None else torch.from_numpy(n).to(DEV) for n in noises]
    d_masked = torch.empty_like(d_pool[0])
    h_masked = torch.empty(d_masked.shape, dtype=d_masked.dtype).pin_memory()
    states = np.array([dfas[0 if row_table is None else row_table[r]][2] for r in range(B)],
                      dtype=np.int32)
    threads = min(oracle.max_threads(), 32)
    emitted = finished = 0
    for t in range(steps):
        k = t % pool
        tokens, _ = dec.step(d_pool[k], noise=d_noise[k], masked_out=d_masked)
        h_masked.copy_(d_masked, non_blocking=True)
        g_tok = tokens.cpu().numpy()
        g_st = dec.states.cpu().numpy()
        g_acc = dec.accept.cpu().numpy()
        torch.cuda.synchronize()
        ref = oracle.step(dfas, vb, vo, pools[k], states, noise=noises[k], row_table=row_table,
                          threads=threads)
        assert np.array_equal(g_tok, ref["tokens"]), "step %d tokens" % t
        assert np.array_equal(g_st, ref["states"]), "step %d states" % t
        assert np.array_equal(g_acc, ref["accept"]), "step %d accept flags" % t
        got = h_masked.view(torch.int16).numpy().view(np.uint16) if w.dtype == "bf16" else h_masked.numpy()
        assert bits_equal(got, ref["masked"]), "step %d masked logits" % t
        states = ref["states"]
        emitted += int((ref["tokens"] >= 0).sum())
        finished = int((states < 0).sum())
    assert emitted > 0
    bad, _ = dec.status()
    assert bad == 0
    return dec, finished


# The five workloads at their own batch sizes and lengths (32 / 256 / 512 / 128 / 64 steps),
# every row compared at every step.

def test_config_api_1k_full_decode():
    decode_and_check("api_1k", pool=32)


def test_config_json_32k_full_decode():
    decode_and_check("json_32k", pool=4)


def test_config_schema40_128k_gumbel_full_decode():
    decode_and_check("schema40_128k", pool=2)


def test_config_string_256k_full_decode():
    _, finished = decode_and_check("string_256k", pool=2)
    assert 0 < finished < 512          # some rows closed their string and stayed finished


def test_config_random10k_mixed_batch_full_decode():
    decode_and_check("random10k_256k", pool=2)


def test_two_calls_share_a_workspace_in_stream_order():
    # scratch is reset by the kernel itself: back-to-back steps on one stream need no host work
    dec, _ = decode_and_check("api_1k", steps=4, pool=4, batch=64)
    assert dec.status()[0] == 0


def test_repeated_runs_are_bit_identical():
    # every kernel twice on the same inputs: any race or order dependence would show
    name = "json_32k"
    dfa = config_dfas(name)[0]
    vb, vo = config_vocab(name)
    V = vo.size - 1
    vocab = cstr.cstr_load_vocab(vb, vo)
    h = cstr.cstr_load_dfa(*dfa)
    S = dfa[0].shape[0]
    t1 = cstr.cstr_table_create(vocab, S)
    t2 = cstr.cstr_table_create(vocab, S)
    cstr.cstr_table_build(t1, h)
    cstr.cstr_table_build(t2, h)
    cstr.cstr_table_build(t2, h)                     # rebuilding over itself changes nothing
    a, b = cstr.cstr_table_download(t1), cstr.cstr_table_download(t2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    B = 64
    logits = to_dev_logits(normal_logits(3, 0, range(B), V, sigma=2.0, dtype="bf16"))
    noise = torch.from_numpy(gumbel_noise(4, 0, range(B), V)).to(DEV)
    ws = cstr.cstr_workspace_create(B)
    outs = []
    for rep in range(3):
        st = torch.full((B,), int(dfa[2]), dtype=torch.int32, device=DEV)
        tok = torch.empty(B, dtype=torch.int32, device=DEV)
        masked = torch.empty_like(logits)
        cstr.cstr_step([t1 if rep else t2], logits, st, tok, masked, ws, noise=noise)
        torch.cuda.synchronize()
        outs.append((tok.cpu().numpy(), st.cpu().numpy(), from_dev_logits(masked)))
    for o in outs[1:]:
        assert all(np.array_equal(x, y) for x, y in zip(outs[0], o))


def test_many_rows_small_vocabulary():
    # more rows than a grid dimension of 65,535 would hold: rows are linearised
    rng = np.random.default_rng(21)
    dfa = dense_random_dfa(rng, 20, live=0.5)
    vb, vo = random_vocab(rng, 96, max_len=3)
    tables = gpu_tables([dfa], vb, vo)
    B, V = 70001, 96
    logits = rng.standard_normal((B, V)).astype(np.float32)
    states = rng.integers(-1, 20, size=B).astype(np.int32)
    run_step_both([dfa], tables, vb, vo, logits, states)


def test_empty_batch_is_a_no_op():
    # zero rows: every step entry point returns without touching anything
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    (table,) = gpu_tables([dfa], vb, vo)
    V = vo.size - 1
    ws = cstr.cstr_workspace_create(4)
    logits = torch.empty((0, V), device=DEV)
    st = torch.empty((0,), dtype=torch.int32, device=DEV)
    cstr.cstr_step([table], logits, st, st.clone(), torch.empty_like(logits), ws)
    cstr.cstr_step_history([table], logits, st, st.clone(), st.clone(), torch.empty_like(logits), ws)
    cstr.cstr_step_static([table], logits, st, st.clone(), torch.empty_like(logits))
    torch.cuda.synchronize()
    assert cstr.cstr_step_status(ws) == (0, 0)


@pytest.mark.parametrize("dtype,gumbel,pinned", [("f32", False, True), ("bf16", True, False)])
def test_step_host_matches_the_oracle(dtype, gumbel, pinned):
    # logits in host memory (pinned or pageable), sliced uploads overlapped with the step
    # kernels: every output as from the oracle, for a batch that does not divide into slices
    dfa = config_dfas("json_32k")[0]
    vb, vo = config_vocab("json_32k")
    V = vo.size - 1
    (table,) = gpu_tables([dfa], vb, vo)
    B = 37
    ws = cstr.cstr_workspace_create(64)
    rng = np.random.default_rng(3)
    states = rng.integers(-1, dfa[0].shape[0], size=B).astype(np.int32)
    for t in range(3):
        logits = normal_logits(9, t, range(B), V, sigma=2.0, dtype=dtype)
        noise = gumbel_noise(1, t, range(B), V) if gumbel else None
        h_logits = torch.from_numpy(logits)
        h_logits = h_logits.view(torch.bfloat16) if dtype == "bf16" else h_logits
        h_noise = None if noise is None else torch.from_numpy(noise)
        if pinned:
            h_logits = h_logits.pin_memory()
        d_states = torch.from_numpy(states).to(DEV)
        h_tok = torch.full((B,), -7, dtype=torch.int32)
        h_st = torch.full((B,), -7, dtype=torch.int32)
        d_logits = torch.empty(h_logits.shape, dtype=h_logits.dtype, device=DEV)
        d_noise = None if noise is None else torch.empty((B, V), device=DEV)
        d_masked = torch.empty_like(d_logits)
        d_tok = torch.empty((B,), dtype=torch.int32, device=DEV)
        d_acc = torch.empty((B,), dtype=torch.uint8, device=DEV)
        h_masked = torch.full(h_logits.shape, 7.0, dtype=h_logits.dtype) if t != 1 else None
        if h_masked is not None and pinned:
            h_masked = h_masked.pin_memory()
        cstr.cstr_step_host([table], h_logits, d_states, h_tok, d_logits, d_masked, d_tok, ws,
                            states_host=h_st, noise_host=h_noise, noise_dev=d_noise, accept_out=d_acc,
                            masked_host=h_masked)
        ref = oracle.step([dfa], vb, vo, logits, states, noise=noise, threads=8)
        assert np.array_equal(h_tok.numpy(), ref["tokens"])          # no synchronisation needed
        assert np.array_equal(h_st.numpy(), ref["states"])
        assert np.array_equal(d_states.cpu().numpy(), ref["states"])
        assert np.array_equal(d_acc.cpu().numpy(), ref["accept"])
        assert bits_equal(from_dev_logits(d_masked), ref["masked"])
        if h_masked is not None:                                     # the host copy, no synchronisation needed
            got = h_masked.view(torch.int16).numpy().view(np.uint16) if dtype == "bf16" else h_masked.numpy()
            assert bits_equal(got, ref["masked"])
        states = ref["states"]
    assert cstr.cstr_step_status(ws)[0] == 0


def test_mixed_batch_with_a_renumbered_table():
    # one sparse automaton (numbered internally: its many-byte states first) beside a dense one
    # and a small one in the same call: every row's state goes into and out of its own table's
    # numbering; fp32 and bf16, with and without noise, a few steps each
    from test_gpu_table import sparse_dfa
    rng = np.random.default_rng(44)
    V = 6000
    vb, vo = random_vocab(rng, V, max_len=8, alphabet=b"abcdefghijklmnopqrstuvwxyz ", empty_prob=0.0)
    dfas = [sparse_dfa(rng, 1500, many_every=29), dense_random_dfa(rng, 700, live=0.6),
            dense_random_dfa(rng, 9, live=0.9)]
    tables = gpu_tables(dfas, vb, vo)
    B = 96
    row_table = rng.integers(0, 3, size=B).astype(np.int32)
    states = np.array([rng.integers(0, dfas[t][0].shape[0]) for t in row_table], dtype=np.int32)
    states[:4] = [3, 32, 61, 1499]                   # many-byte and picky states of the sparse one
    row_table[:4] = 0
    for dtype in ("f32", "bf16"):
        st = states.copy()
        for t in range(4):
            logits = rand_logits(rng, B, V, V, dtype)
            noise = None
            if t % 2:
                noise = -np.log(-np.log(rng.random((B, V)))).astype(np.float32)
            ref = run_step_both(dfas, tables, vb, vo, logits, st, noise=noise, row_table=row_table)
            st = ref["states"]
            st[st < 0] = 0                           # keep rows going
