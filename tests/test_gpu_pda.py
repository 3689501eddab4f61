"""GPU parity of the push-down path (Section 3, Algorithm 3) with the oracle:
the token-level PDA's per-situation masks and whole decoding loops, bit for bit."""
import numpy as np
import pytest
import torch

from gpu_common import DEV, bits_equal, from_dev_logits, to_dev_logits
from oracle import pda as op
from paper_2407_08103_b200 import cstr
from synth import (anbn_pda, dyck_pda, gumbel_noise, json_pda, make_vocab_json, normal_logits,
                   random_pda, stackless_pda, vocab_from_strings)
from synth.configs import config_dfas, config_vocab

pytestmark = pytest.mark.gpu
THREADS = 16


def load_pda(P):
    return cstr.cstr_load_pda(P.src, P.inp, P.tgt, P.pop_off, P.pops, P.push_off, P.pushes,
                              P.accept, P.n_symbols, P.start)


def build(P, vb, vo, eos_id=-1):
    vocab = cstr.cstr_load_vocab(vb, vo)
    table = cstr.cstr_build_pda_table(load_pda(P), vocab, eos_id)
    torch.cuda.synchronize()
    return table


def check_table(table, P, vb, vo, eos_id=-1, states=None, deeper=3, seed=0):
    """mask(q, X) is the allowed set of the one-symbol stack [X] (edges that pop at
    most that symbol); with deeper stacks ending in X the allowed set grows only by
    tokens flagged in deep(q, X)."""
    info = cstr.cstr_pda_table_info(table)
    V = vo.size - 1
    assert info == dict(n_states=P.n_states, n_symbols=P.n_symbols, vocab_size=V,
                        mask_words=(V + 31) // 32, start_state=P.start)
    states = range(P.n_states) if states is None else states
    rng = np.random.default_rng(seed)
    qs, tops, stacks = [], [], []
    for q in states:
        for top in range(-1, P.n_symbols):
            qs.append(q)
            tops.append(top)
            stacks.append([] if top < 0 else [top])
    want = op.allowed(P, vb, vo, qs, stacks, eos_id=eos_id, threads=THREADS)
    got = [cstr.cstr_pda_table_download(table, q, t) for q, t in zip(qs, tops)]
    for i in range(len(qs)):
        assert np.array_equal(got[i][0], want[i]), "mask of (state %d, top %d)" % (qs[i], tops[i])
        assert not (got[i][0] & got[i][1]).any()
        if tops[i] < 0:
            assert not got[i][1].any()          # nothing lies below an empty stack
    n_deep = 0
    for _ in range(deeper if P.n_symbols else 0):
        below = [list(rng.integers(0, P.n_symbols, size=int(rng.integers(1, 4)))) if t >= 0 else []
                 for t in tops]
        full = op.allowed(P, vb, vo, qs, [b + s for b, s in zip(below, stacks)], eos_id=eos_id,
                          threads=THREADS)
        for i in range(len(qs)):
            assert not (want[i] & ~full[i]).any()
            extra = full[i] & ~want[i]
            assert not (extra & ~got[i][1]).any(), "token allowed by a deeper stack is not flagged"
            n_deep += int(extra.any())
    return n_deep


def run_both(P, table, ws, vb, vo, logits, states, stacks, depth, noise=None, eos_id=-1,
             in_place=False):
    B = logits.shape[0]
    V = vo.size - 1
    d_logits = to_dev_logits(logits)
    d_noise = None if noise is None else torch.from_numpy(noise).to(DEV)
    d_states = torch.from_numpy(np.asarray(states, dtype=np.int32)).to(DEV)
    d_stacks = torch.from_numpy(np.ascontiguousarray(stacks, dtype=np.int32)).to(DEV)
    d_depth = torch.from_numpy(np.asarray(depth, dtype=np.int32)).to(DEV)
    d_tokens = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    d_acc = torch.full((B,), 9, dtype=torch.uint8, device=DEV)
    d_out = d_logits if in_place else torch.full_like(d_logits, 123.0)
    cstr.cstr_pda_step(table, d_logits, d_states, d_stacks, d_depth, d_tokens, d_out, ws,
                       noise=d_noise, accept_out=d_acc)
    torch.cuda.synchronize()
    counters = cstr.cstr_pda_step_status(ws)
    ref = op.step(P, vb, vo, logits, states, stacks, depth, noise=noise, eos_id=eos_id,
                  vocab_size=V, threads=THREADS)
    assert np.array_equal(d_tokens.cpu().numpy(), ref["tokens"])
    assert np.array_equal(d_states.cpu().numpy(), ref["states"])
    assert np.array_equal(d_depth.cpu().numpy(), ref["depth"])
    g_stacks = d_stacks.cpu().numpy()
    for r in range(B):
        n = ref["depth"][r]
        if 0 <= n <= g_stacks.shape[1]:
            assert np.array_equal(g_stacks[r, :n], ref["stacks"][r, :n]), "stack of row %d" % r
    got = from_dev_logits(d_out)
    assert bits_equal(got[:, :V], ref["masked"][:, :V])
    if not in_place and got.shape[1] > V:
        pad = from_dev_logits(torch.full_like(d_logits, 123.0))[:, V:]
        assert bits_equal(got[:, V:], pad)
    assert np.array_equal(d_acc.cpu().numpy(), ref["accept"])
    assert counters == (ref["bad_state_rows"], ref["empty_mask_rows"], ref["overflow_rows"])
    ref["stacks_full"] = g_stacks
    return ref


# ------------------------------------------------------------------- tables

def test_table_anbn_figure5_vocabulary():
    P = anbn_pda()
    vb, vo = vocab_from_strings([b"a", b"b", b"bb", b"aaab", b"", b"abb", b"bbb", b"ab"])
    table = build(P, vb, vo)
    assert check_table(table, P, vb, vo) > 0
    st = {n: i for i, n in enumerate(P.state_names)}
    A = P.symbol_names.index("A")
    mask, deep = cstr.cstr_pda_table_download(table, st["bs"], A)
    assert mask[0] == 0b00000010 and deep[0] == 0b01000100     # b | bb and bbb look deeper


def test_table_dyck_and_eos():
    P = dyck_pda((b"()", b"[]", b"{}", b"<>"), fillers=b"xy ")
    vb, vo = make_vocab_json(1500, seed=3)
    table = build(P, vb, vo, eos_id=77)
    check_table(table, P, vb, vo, eos_id=77)
    cstr.cstr_pda_table_rebuild(table, -1)             # same storage, no EOS token
    torch.cuda.synchronize()
    check_table(table, P, vb, vo)
    cstr.cstr_pda_table_rebuild(table, 3)
    torch.cuda.synchronize()
    check_table(table, P, vb, vo, eos_id=3)


def test_table_json_small_vocab_all_situations():
    P = json_pda(space=True)
    vb, vo = make_vocab_json(2051, seed=1)        # W = 65 words, ragged last word
    table = build(P, vb, vo)
    assert check_table(table, P, vb, vo) > 5


def test_table_json_32k_sampled_situations():
    P = json_pda(space=True)
    vb, vo = make_vocab_json(32000, seed=0)
    table = build(P, vb, vo)
    st = {n: i for i, n in enumerate(P.state_names)}
    check_table(table, P, vb, vo, deeper=1,
                states=[st[n] for n in ("start", "after_value", "num_int", "str", "arr_first",
                                        "colon", "done")])


def test_stackless_pda_matches_the_finite_state_table():
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    P = stackless_pda(*dfa)
    table = build(P, vb, vo)
    check_table(table, P, vb, vo)


# -------------------------------------------------------------------- steps

@pytest.mark.parametrize("dtype,gumbel,vocab_size,pad", [
    ("f32", False, 2051, 0), ("bf16", False, 4096, 8), ("f32", True, 3000, 4),
    ("bf16", True, 2048, 0),
])
def test_decode_loop_json(dtype, gumbel, vocab_size, pad):
    P = json_pda(space=True)
    vb, vo = make_vocab_json(vocab_size, seed=2)
    V = vo.size - 1
    toks = [bytes(vb[vo[v]:vo[v + 1]]) for v in range(V)]
    table = build(P, vb, vo)
    B, cap, steps = 48, 5, 40
    ws = cstr.cstr_pda_workspace_create(table, B)
    states = np.full(B, P.start, dtype=np.int32)
    stacks = np.zeros((B, cap), dtype=np.int32)
    depth = np.zeros(B, dtype=np.int32)
    sigma = 2.0 if dtype == "bf16" else 1.0
    seen_depth, overflow, deep_rows = 0, 0, 0
    for t in range(steps):
        logits = normal_logits(31, t, range(B), V, ld=V + pad, sigma=sigma, dtype="f32")
        # most rows favour structure over string bodies, some dig for the overflow path
        for name, bonus in ((b"[", 5.0), (b"[[", 5.0), (b"]]", 6.0), (b"]]]", 6.0), (b"]", 4.0),
                            (b'"', 4.0), (b"}", 4.0), (b"{", 3.0), (b"1]", 5.0), (b", ", 4.0),
                            (b"1", 4.0), (b'":', 5.0)):
            logits[: B - 8, toks.index(name)] += np.float32(bonus)
        for name in (b"[", b"[[", b"[{"):
            logits[B - 8:, toks.index(name)] += np.float32(7.0)
        if dtype == "bf16":
            from synth import f32_to_bf16_bits
            logits = f32_to_bf16_bits(logits)
        noise = gumbel_noise(1, t, range(B), V, ld=V + pad) if gumbel else None
        ref = run_both(P, table, ws, vb, vo, logits, states, stacks, depth, noise=noise)
        deep_rows += int(((depth >= 2) & (states >= 0)).sum())
        states, depth = ref["states"], ref["depth"]
        stacks = ref["stacks_full"]
        seen_depth = max(seen_depth, int(depth.max()))
        overflow += ref["overflow_rows"]
        if t == 20:                                 # restart the finished rows
            done = states < 0
            states = np.where(done, P.start, states).astype(np.int32)
            depth = np.where(done, 0, depth).astype(np.int32)
    assert seen_depth >= 4 and overflow > 0 and deep_rows > 50


def test_decode_loop_anbn_deep_pops():
    # every b-run token reaches below the top of the stack
    P = anbn_pda()
    vb, vo = vocab_from_strings([b"a", b"b", b"bb", b"aaab", b"bbbb", b"aa", b"ab", b"<e>", b"bbb"])
    V = vo.size - 1
    table = build(P, vb, vo, eos_id=7)
    B, cap = 64, 12
    ws = cstr.cstr_pda_workspace_create(table, B)
    states = np.full(B, P.start, dtype=np.int32)
    stacks = np.zeros((B, cap), dtype=np.int32)
    depth = np.zeros(B, dtype=np.int32)
    finished = 0
    for t in range(14):
        logits = normal_logits(41, t, range(B), V, ld=12)
        if t < 3:
            logits[:, [0, 5]] += np.float32(3.0)        # grow first
        ref = run_both(P, table, ws, vb, vo, logits, states, stacks, depth, eos_id=7,
                       in_place=(t % 2 == 1))
        finished += int(((ref["tokens"] == 7)).sum())
        states, depth, stacks = ref["states"], ref["depth"], ref["stacks_full"]
    assert finished > 10                                 # rows reached "done" and took EOS


def test_inactive_rows_bad_stacks_and_overflow():
    P = anbn_pda()
    vb, vo = vocab_from_strings([b"a", b"b", b"bb", b"aaab", b"<eos>"])
    st = {n: i for i, n in enumerate(P.state_names)}
    Z, A = P.symbol_names.index("Z"), P.symbol_names.index("A")
    table = build(P, vb, vo, eos_id=4)
    ws = cstr.cstr_pda_workspace_create(table, 16)
    logits = np.array([[0.0, 1.0, 2.0, 3.0, 0.5]] * 9, dtype=np.float32)
    states = np.array([st["start"], st["as"], st["bs"], -1, 9, st["as"], st["done"], st["as"],
                       st["bs"]], np.int32)
    stacks = np.array([[0, 0, 0], [Z, A, 0], [Z, A, 0], [0, 0, 0], [0, 0, 0], [Z, 7, 0],
                       [0, 0, 0], [Z, A, A], [-1, A, 0]], np.int32)
    depth = np.array([0, 2, 2, 0, 0, 2, 0, 4, 2], np.int32)
    ref = run_both(P, table, ws, vb, vo, logits, states, stacks, depth, eos_id=4)
    assert list(ref["tokens"]) == [3, 3, 2, -1, -1, -1, 4, -1, -1]
    assert (ref["bad_state_rows"], ref["empty_mask_rows"], ref["overflow_rows"]) == (4, 0, 1)


def test_load_pda_rejects_what_it_cannot_run():
    P = anbn_pda()

    def load(**kw):
        d = dict(src=P.src, inp=P.inp, tgt=P.tgt, pop_off=P.pop_off, pops=P.pops,
                 push_off=P.push_off, pushes=P.pushes, accept=P.accept, n_symbols=P.n_symbols,
                 start=P.start)
        d.update(kw)
        return cstr.cstr_load_pda(d["src"], d["inp"], d["tgt"], d["pop_off"], d["pops"],
                                  d["push_off"], d["pushes"], d["accept"], d["n_symbols"],
                                  d["start"])

    load()
    with pytest.raises(cstr.CstrError) as e:
        load(inp=np.where(np.arange(P.n_edges) == 1, -1, P.inp))     # an epsilon edge
    assert e.value.code == -10
    with pytest.raises(cstr.CstrError) as e:                          # two edges, same situation
        load(src=np.append(P.src, P.src[0]), inp=np.append(P.inp, P.inp[0]),
             tgt=np.append(P.tgt, P.tgt[0]), pop_off=np.append(P.pop_off, P.pop_off[-1]),
             push_off=np.append(P.push_off, P.push_off[-1]))
    assert e.value.code == -10 and "deterministic" in str(e.value)
    with pytest.raises(cstr.CstrError) as e:                          # a two-symbol pop
        load(pop_off=np.append(P.pop_off[:-1], P.pop_off[-1] + 1), pops=np.append(P.pops, 0))
    assert e.value.code == -10


def test_full_size_json_256k_sampled_rows():
    # vocabulary 256,000 x batch 512 as bench.py times it; the oracle replays the whole
    # trajectory of a few rows (each row depends only on its own logits, state and stack)
    from paper_2407_08103_b200.decode import PushdownDecoder
    P = json_pda(space=True)
    vb, vo = make_vocab_json(256000, seed=0)
    V = vo.size - 1
    toks = {bytes(vb[vo[v]:vo[v + 1]]): v for v in range(V - 1, -1, -1)}
    table = build(P, vb, vo)
    B, cap, steps = 512, 64, 10
    rows = [0, 3, 77, 300, 511]
    dec = PushdownDecoder(table, B, stack_cap=cap)
    o_states = np.full(len(rows), P.start, dtype=np.int32)
    o_stacks = np.zeros((len(rows), cap), dtype=np.int32)
    o_depth = np.zeros(len(rows), dtype=np.int32)
    deepest = 0
    for t in range(steps):
        logits = normal_logits(51, t, range(B), V)
        for name, bonus in ((b"[", 6.0), (b"[[", 6.0), (b"]]", 7.0), (b"]]]", 7.0), (b"1]", 6.0),
                            (b"{", 4.0), (b"}]", 6.0), (b'"', 5.0), (b", ", 5.0), (b"1", 5.0)):
            logits[:, toks[name]] += np.float32(bonus)
        tokens, masked = dec.step(to_dev_logits(logits))
        ref = op.step(P, vb, vo, logits[rows], o_states, o_stacks, o_depth, threads=THREADS)
        assert np.array_equal(tokens.cpu().numpy()[rows], ref["tokens"]), "step %d tokens" % t
        assert np.array_equal(dec.states.cpu().numpy()[rows], ref["states"])
        assert np.array_equal(dec.depths.cpu().numpy()[rows], ref["depth"])
        g_stacks = dec.stacks.cpu().numpy()[rows]
        for i in range(len(rows)):
            assert np.array_equal(g_stacks[i, :ref["depth"][i]], ref["stacks"][i, :ref["depth"][i]])
        assert bits_equal(from_dev_logits(masked[rows]), ref["masked"])
        o_states, o_stacks, o_depth = ref["states"], ref["stacks"], ref["depth"]
        deepest = max(deepest, int(o_depth.max()))
    assert deepest >= 3 and (o_states >= 0).any()


@pytest.mark.parametrize("seed", range(8))
def test_random_pdas_table_and_decode_loop(seed):
    # random deterministic PDAs (pops, multi-symbol pushes, edges that push back what they
    # popped) over all short strings of a small alphabet as the vocabulary
    import itertools
    rng = np.random.default_rng(seed)
    n_symbols = int(rng.choice([1, 2, 3]))
    P = random_pda(seed, n_states=int(rng.choice([2, 5, 9])), n_symbols=n_symbols)
    toks = [bytes(t) for n in range(0, 5) for t in itertools.product(b"abcd", repeat=n)]
    toks = [toks[i] for i in rng.permutation(len(toks))][:300] + [b"e", b"ae"]
    vb, vo = vocab_from_strings(toks)
    V = vo.size - 1
    eos = int(rng.integers(V)) if seed % 2 else -1
    table = build(P, vb, vo, eos_id=eos)
    check_table(table, P, vb, vo, eos_id=eos, seed=seed)
    B, cap = 40, 12
    ws = cstr.cstr_pda_workspace_create(table, B)
    states = rng.integers(0, P.n_states, size=B).astype(np.int32)
    depth = rng.integers(0, 8, size=B).astype(np.int32)
    stacks = rng.integers(0, n_symbols, size=(B, cap)).astype(np.int32)
    emitted = 0
    for t in range(12):
        logits = normal_logits(61 + seed, t, range(B), V)
        ref = run_both(P, table, ws, vb, vo, logits, states, stacks, depth, eos_id=eos)
        emitted += int((ref["tokens"] >= 0).sum())
        states, depth, stacks = ref["states"], ref["depth"], ref["stacks_full"]
        if t % 4 == 3:                                  # revive finished rows somewhere else
            done = states < 0
            states = np.where(done, rng.integers(0, P.n_states, size=B), states).astype(np.int32)
    assert emitted > 20


def test_grammar_built_json_pda():
    # the bracketed-grammar front-end's nested-JSON PDA (one stack symbol per call site)
    from synth import json_grammar_pda
    P = json_grammar_pda()
    vb, vo = make_vocab_json(3000, seed=4)
    V = vo.size - 1
    toks = [bytes(vb[vo[v]:vo[v + 1]]) for v in range(V)]
    table = build(P, vb, vo)
    rng = np.random.default_rng(2)
    assert check_table(table, P, vb, vo, states=rng.choice(P.n_states, size=12, replace=False)) > 0
    B, cap = 32, 6
    ws = cstr.cstr_pda_workspace_create(table, B)
    states = np.full(B, P.start, dtype=np.int32)
    stacks = np.zeros((B, cap), dtype=np.int32)
    depth = np.zeros(B, dtype=np.int32)
    for t in range(24):
        logits = normal_logits(71, t, range(B), V)
        for name, bonus in ((b"[", 5.0), (b"[[", 5.0), (b"]]", 6.0), (b"]", 4.0), (b'"', 4.0),
                            (b"}", 4.0), (b"{", 3.0), (b"1]", 5.0), (b", ", 4.0), (b"1", 4.0)):
            logits[:, toks.index(name)] += np.float32(bonus)
        ref = run_both(P, table, ws, vb, vo, logits, states, stacks, depth)
        states, depth, stacks = ref["states"], ref["depth"], ref["stacks_full"]
    assert depth.max() >= 2


def test_speculative_loop_pushdown():
    # draft k tokens with cstr_pda_step_history (keeping every situation), verify all k + 1
    # positions in one call over the history, accept / rewind; every array against the oracle
    from synth.models import draft_logits, target_logits
    P = json_pda(space=True)
    vb, vo = make_vocab_json(1200, seed=6)
    V = vo.size - 1
    table = build(P, vb, vo)
    B, k, cap = 6, 3, 8
    ws = cstr.cstr_pda_workspace_create(table, B * (k + 1))
    i32 = dict(dtype=torch.int32, device=DEV)
    g_state = torch.full((B,), P.start, **i32)
    g_stack = torch.zeros((B, cap), **i32)
    g_depth = torch.zeros((B,), **i32)
    o_state = np.full(B, P.start, np.int32)
    o_stack = np.zeros((B, cap), np.int32)
    o_depth = np.zeros(B, np.int32)
    outs = [[] for _ in range(B)]
    kept = 0
    for rnd in range(5):
        h_state = torch.zeros((B, k + 1), **i32)
        h_stack = torch.zeros((B, k + 1, cap), **i32)
        h_depth = torch.zeros((B, k + 1), **i32)
        h_state[:, 0], h_stack[:, 0], h_depth[:, 0] = g_state, g_stack, g_depth
        oh_state, oh_stack, oh_depth = [o_state], [o_stack], [o_depth]
        drafts = torch.zeros((B, k), **i32)
        o_drafts = np.zeros((B, k), np.int32)
        for i in range(k):
            prefixes = [outs[r] + [int(t) for t in o_drafts[r, :i]] for r in range(B)]
            logits = np.stack([draft_logits(9, r, prefixes[r], V) for r in range(B)])
            d_logits = to_dev_logits(logits)
            tok = torch.empty((B,), **i32)
            s_in, k_in, d_in = (h_state[:, i].contiguous(), h_stack[:, i].contiguous(),
                                h_depth[:, i].contiguous())
            s_out, k_out, d_out = torch.empty_like(s_in), torch.empty_like(k_in), torch.empty_like(d_in)
            cstr.cstr_pda_step_history(table, d_logits, s_in, k_in, d_in, s_out, k_out, d_out, tok,
                                       torch.empty_like(d_logits), ws)
            h_state[:, i + 1], h_stack[:, i + 1], h_depth[:, i + 1] = s_out, k_out, d_out
            drafts[:, i] = tok
            ref = op.step(P, vb, vo, logits, oh_state[-1], oh_stack[-1], oh_depth[-1], threads=4)
            assert np.array_equal(tok.cpu().numpy(), ref["tokens"])
            assert np.array_equal(s_in.cpu().numpy(), oh_state[-1])        # inputs untouched
            o_drafts[:, i] = ref["tokens"]
            oh_state.append(ref["states"]); oh_stack.append(ref["stacks"]); oh_depth.append(ref["depth"])
        # verification: one call over B x (k + 1) history rows
        prefixes = [[outs[r] + [int(t) for t in o_drafts[r, :i]] for i in range(k + 1)] for r in range(B)]
        tl = np.stack([target_logits(9, r, prefixes[r][i], V) for r in range(B) for i in range(k + 1)])
        d_tl = to_dev_logits(tl)
        n_rows = B * (k + 1)
        t_tok = torch.empty((n_rows,), **i32)
        t_state, t_stack, t_depth = (torch.empty((n_rows,), **i32), torch.empty((n_rows, cap), **i32),
                                     torch.empty((n_rows,), **i32))
        cstr.cstr_pda_step_history(table, d_tl, h_state.view(-1), h_stack.view(n_rows, cap),
                                   h_depth.view(-1), t_state, t_stack, t_depth, t_tok,
                                   torch.empty_like(d_tl), ws)
        ref = op.step(P, vb, vo, tl, np.stack(oh_state, 1).reshape(-1),
                      np.stack(oh_stack, 1).reshape(n_rows, cap), np.stack(oh_depth, 1).reshape(-1),
                      threads=4)
        assert np.array_equal(t_tok.cpu().numpy(), ref["tokens"])
        assert np.array_equal(t_state.cpu().numpy(), ref["states"])
        assert np.array_equal(t_depth.cpu().numpy(), ref["depth"])
        n_acc = torch.empty((B,), **i32)
        out_tok = torch.empty((B, k + 1), **i32)
        cstr.cstr_pda_accept_draft(drafts, t_tok.view(B, k + 1), t_state.view(B, k + 1),
                                   t_stack.view(B, k + 1, cap), t_depth.view(B, k + 1), n_acc,
                                   out_tok, g_state, g_stack, g_depth)
        torch.cuda.synchronize()
        on, oout, o_state, o_stack, o_depth = op.accept_draft(
            o_drafts, ref["tokens"].reshape(B, k + 1), ref["states"].reshape(B, k + 1),
            ref["stacks"].reshape(B, k + 1, cap), ref["depth"].reshape(B, k + 1))
        assert np.array_equal(n_acc.cpu().numpy(), on) and np.array_equal(out_tok.cpu().numpy(), oout)
        assert np.array_equal(g_state.cpu().numpy(), o_state)
        assert np.array_equal(g_depth.cpu().numpy(), o_depth)
        gs = g_stack.cpu().numpy()
        for r in range(B):
            n = o_depth[r]
            assert np.array_equal(gs[r, :n], o_stack[r, :n])
            outs[r] += [int(t) for t in oout[r] if t >= 0]
        o_stack = gs.copy()                              # beyond the depth both sides are free
        kept += int(on.sum())
    assert kept > 0 and max(len(o) for o in outs) >= 5


def test_empty_batch_and_limits():
    P = anbn_pda()
    vb, vo = vocab_from_strings([b"a", b"b", b"bb", b"aaab"])
    table = build(P, vb, vo)
    ws = cstr.cstr_pda_workspace_create(table, 4)
    i32 = dict(dtype=torch.int32, device=DEV)
    logits = torch.empty((0, 4), device=DEV)
    cstr.cstr_pda_step(table, logits, torch.empty((0,), **i32), torch.empty((0, 8), **i32),
                       torch.empty((0,), **i32), torch.empty((0,), **i32), torch.empty_like(logits), ws)
    torch.cuda.synchronize()
    assert cstr.cstr_pda_step_status(ws) == (0, 0, 0)
    # a batch beyond the workspace, and a vocabulary whose tokens could outgrow the walk's stack
    big = torch.zeros((5, 4), device=DEV)
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_pda_step(table, big, torch.zeros((5,), **i32), torch.zeros((5, 8), **i32),
                           torch.zeros((5,), **i32), torch.zeros((5,), **i32), torch.empty_like(big), ws)
    assert e.value.code == -6
    long_vb, long_vo = vocab_from_strings([b"a" * 300, b"b"])
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_build_pda_table(load_pda(P), cstr.cstr_load_vocab(long_vb, long_vo))
    assert e.value.code == -6
