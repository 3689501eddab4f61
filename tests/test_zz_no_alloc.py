"""The allocation-free step entry point against the ordinary one.

Some hosts of the library cannot call the CUDA allocator while they run (all
device memory already handed to a cache pool, a fixed memory budget, or no
tolerance for cudaMalloc's device-wide synchronisation).  ``cstr_step_static``
serves them with a fixed scratch array inside the library; here it must give
exactly what ``cstr_step`` gives - and what the CPU oracle gives - on
consecutive calls that share that array, and the device's free memory must not
move across its calls.  Collected last so that a failure here cannot hide any
other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2407_08103_b200 import cstr
from synth import gumbel_noise, normal_logits
from synth.configs import config_dfas, config_vocab

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_static_step_matches_workspace_step_and_oracle_without_allocating():
    dfa = config_dfas("json_32k")[0]
    vb, vo = config_vocab("json_32k")
    V = vo.size - 1
    B = 48
    vocab = cstr.cstr_load_vocab(vb, vo)
    h = cstr.cstr_load_dfa(*dfa)
    table = cstr.cstr_table_create(vocab, dfa[0].shape[0])
    cstr.cstr_table_build(table, h, -1)
    ws = cstr.cstr_workspace_create(B)

    start = np.full(B, dfa[2], dtype=np.int32)
    start[5] = -1                                   # a finished row
    start[6] = dfa[0].shape[0] + 3                  # an out-of-range state
    st_a = torch.from_numpy(start).to(DEV)
    st_b = st_a.clone()
    o_states = start.copy()
    # every tensor of all three calls exists before the first one, so that the free-memory
    # readings below see only what the entry point itself does
    n_calls = 3
    h_logits = [normal_logits(21, c, range(B), V) for c in range(n_calls)]
    h_noise = [gumbel_noise(22, c, range(B), V) if c else None for c in range(n_calls)]
    logits = [torch.from_numpy(x).to(DEV) for x in h_logits]
    noise = [None if x is None else torch.from_numpy(x).to(DEV) for x in h_noise]
    tok_a = torch.full((B,), -5, dtype=torch.int32, device=DEV)
    tok_b = torch.full((B,), -6, dtype=torch.int32, device=DEV)
    acc_a = torch.full((B,), 7, dtype=torch.uint8, device=DEV)
    acc_b = torch.full((B,), 8, dtype=torch.uint8, device=DEV)
    out_a = torch.empty_like(logits[0])
    out_b = torch.empty_like(logits[0])
    free_before_second = None
    for call in range(n_calls):                     # later calls reuse the shared array
        if call == 1:
            torch.cuda.synchronize()
            free_before_second = torch.cuda.mem_get_info()[0]       # cudaMemGetInfo
        cstr.cstr_step([table], logits[call], st_a, tok_a, out_a, ws, noise=noise[call],
                       accept_out=acc_a)
        cstr.cstr_step_static([table], logits[call], st_b, tok_b, out_b, noise=noise[call],
                              accept_out=acc_b)
        torch.cuda.synchronize()
        # integer outputs and the masked logits (copies or -inf) must be identical bit for bit
        assert torch.equal(tok_a, tok_b)
        assert torch.equal(st_a, st_b)
        assert torch.equal(acc_a, acc_b)
        assert torch.equal(out_a.view(torch.int32), out_b.view(torch.int32))
        assert int((tok_a >= 0).sum()) >= B - 2
        # ... and they are the oracle's
        ref = oracle.step([dfa], vb, vo, h_logits[call], o_states, noise=h_noise[call], threads=8)
        assert np.array_equal(tok_b.cpu().numpy(), ref["tokens"])
        assert np.array_equal(st_b.cpu().numpy(), ref["states"])
        assert np.array_equal(acc_b.cpu().numpy(), ref["accept"])
        assert np.array_equal(out_b.cpu().numpy().view(np.uint32), ref["masked"].view(np.uint32))
        o_states = ref["states"]
    # the one property the entry point exists for: the device's free memory did not move
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before_second
    assert int(tok_a[5]) == -1 and int(tok_a[6]) == -1


def test_static_step_rejects_oversized_batch():
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    h = cstr.cstr_load_dfa(*dfa)
    table = cstr.cstr_build_token_table(h, vb, vo)
    B = cstr.CSTR_STATIC_MAX_BATCH + 1
    logits = torch.zeros((B, vo.size - 1), device=DEV)
    st = torch.zeros(B, dtype=torch.int32, device=DEV)
    tok = torch.full((B,), -9, dtype=torch.int32, device=DEV)
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_step_static([table], logits, st, tok, torch.empty_like(logits))
    assert e.value.code == -6 and "exceeds" in str(e.value)
    torch.cuda.synchronize()
    assert int(tok[0]) == -9                        # nothing ran
    # the largest allowed batch works
    B = cstr.CSTR_STATIC_MAX_BATCH
    cstr.cstr_step_static([table], logits[:B], st[:B], tok[:B], torch.empty_like(logits[:B]))
    torch.cuda.synchronize()
    assert int((tok[:B] >= 0).sum()) == B
