"""GPU parity for the rewindable constraint: state-history step, batched target
verification over the history, accept / rewind - against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_08103_b200 import cstr
from synth.configs import config_dfas, config_vocab
from synth.models import draft_logits, target_logits

from gpu_common import DEV, bits_equal, gpu_tables

pytestmark = pytest.mark.gpu


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


def test_accept_draft_random():
    rng = np.random.default_rng(0)
    for B, k in ((1, 0), (5, 1), (300, 4), (64, 7)):
        draft = rng.integers(-1, 4, size=(B, k)).astype(np.int32)
        tgt = rng.integers(-1, 4, size=(B, k + 1)).astype(np.int32)
        tgt[: B // 2, :k] = draft[: B // 2]              # half the rows accept everything
        st = rng.integers(-1, 50, size=(B, k + 1)).astype(np.int32)
        n_o, out_o, s_o = oracle.accept_draft(draft, tgt, st)
        n = torch.full((B,), -9, dtype=torch.int32, device=DEV)
        out = torch.full((B, k + 1), -9, dtype=torch.int32, device=DEV)
        s = torch.full((B,), -9, dtype=torch.int32, device=DEV)
        cstr.cstr_accept_draft(dev_i32(draft).reshape(B, k), dev_i32(tgt), dev_i32(st), n, out, s)
        torch.cuda.synchronize()
        assert np.array_equal(n.cpu().numpy(), n_o)
        assert np.array_equal(out.cpu().numpy(), out_o)
        assert np.array_equal(s.cpu().numpy(), s_o)


def test_speculative_loop_matches_oracle():
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    V = vo.size - 1
    (table,) = gpu_tables([dfa], vb, vo)
    B, k, seed = 6, 4, 31
    ws_draft = cstr.cstr_workspace_create(B)
    ws_verify = cstr.cstr_workspace_create(B * (k + 1))
    prefixes = [[] for _ in range(B)]
    state = np.full(B, dfa[2], dtype=np.int32)
    d_state = dev_i32(state)
    for rnd in range(6):
        # ---- draft k tokens, keeping the state history on the device: hist[i] = q_i
        hist = torch.empty((k + 1, B), dtype=torch.int32, device=DEV)
        hist[0].copy_(d_state)
        d_draft = torch.empty((k, B), dtype=torch.int32, device=DEV)
        o_hist, o_draft = [state.copy()], []
        for i in range(k):
            lg = np.stack([draft_logits(seed, r, prefixes[r] + [int(t[r]) for t in o_draft], V)
                           for r in range(B)])
            d_lg = torch.from_numpy(lg).to(DEV)
            cstr.cstr_step_history([table], d_lg, hist[i], hist[i + 1], d_draft[i],
                                   torch.empty_like(d_lg), ws_draft)
            ref = oracle.step([dfa], vb, vo, lg, o_hist[-1])
            o_draft.append(ref["tokens"])
            o_hist.append(ref["states"])
        torch.cuda.synchronize()
        assert np.array_equal(hist.cpu().numpy(), np.stack(o_hist))          # inputs untouched, history exact
        assert np.array_equal(d_draft.cpu().numpy(), np.stack(o_draft))
        # ---- verify: one step over B x (k + 1) rows, states = the history, row-major by sequence
        draft_bk = np.stack(o_draft, axis=1)                                  # [B][k]
        tl = np.stack([target_logits(seed, r, prefixes[r] + [int(t) for t in draft_bk[r, :i]], V)
                       for r in range(B) for i in range(k + 1)])
        flat_states = hist.t().contiguous().reshape(-1)                       # [B][k + 1]
        d_tl = torch.from_numpy(tl).to(DEV)
        t_tok = torch.empty(B * (k + 1), dtype=torch.int32, device=DEV)
        t_st = torch.empty(B * (k + 1), dtype=torch.int32, device=DEV)
        t_masked = torch.empty_like(d_tl)
        cstr.cstr_step_history([table], d_tl, flat_states, t_st, t_tok, t_masked, ws_verify)
        ref = oracle.step([dfa], vb, vo, tl, np.stack(o_hist, axis=1).reshape(-1))
        torch.cuda.synchronize()
        assert np.array_equal(t_tok.cpu().numpy(), ref["tokens"])
        assert np.array_equal(t_st.cpu().numpy(), ref["states"])
        assert bits_equal(t_masked.cpu().numpy(), ref["masked"])              # penalised target logits
        # ---- accept / rewind
        n = torch.empty(B, dtype=torch.int32, device=DEV)
        out = torch.empty((B, k + 1), dtype=torch.int32, device=DEV)
        cstr.cstr_accept_draft(d_draft.t().contiguous(), t_tok.reshape(B, k + 1),
                               t_st.reshape(B, k + 1), n, out, d_state)
        n_o, out_o, s_o = oracle.accept_draft(draft_bk, ref["tokens"].reshape(B, k + 1),
                                              ref["states"].reshape(B, k + 1))
        torch.cuda.synchronize()
        assert np.array_equal(n.cpu().numpy(), n_o)
        assert np.array_equal(out.cpu().numpy(), out_o)
        assert np.array_equal(d_state.cpu().numpy(), s_o)
        state = s_o
        for r in range(B):
            prefixes[r] += [int(t) for t in out_o[r] if t >= 0]
    assert max(len(p) for p in prefixes) >= 6
