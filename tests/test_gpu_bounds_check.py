"""The small parity cases once more, against the checking build of the library.

``libcstr_check.so`` is the same source compiled with ``-DCSTR_BOUNDS_CHECK``: every index a
kernel forms into the DFA table, the token table, the ballot rows, the vocabulary arrays, the
logits and the push-down tables is compared with its array's extent; an index outside is
counted in a record on the device and the access skipped (no trap).  The memory checker of
the CUDA toolkit is not available where these tests run, so this build and the bit-exact
comparison with the oracle are the memory-safety evidence: each case below must reproduce
the oracle AND leave the record at zero.
"""
import pytest
import torch

from paper_2407_08103_b200 import cstr

import test_gpu_pda as pda_cases
import test_gpu_speculative as spec_cases
import test_gpu_step as step_cases
import test_gpu_table as table_cases
import test_gpu_terminals as term_cases

pytestmark = pytest.mark.gpu


@pytest.fixture
def checked():
    cstr.use_check_library(True)
    try:
        cstr.cstr_debug_bounds_status(reset=True)
        yield
        torch.cuda.synchronize()
        record = cstr.cstr_debug_bounds_status(reset=True)
        assert record[0] == 0, "out-of-range index: site %d, index %d, extent %d" % record[1:]
    finally:
        cstr.use_check_library(False)


def test_the_record_works(checked):
    # the checking build is the one in use, and its record starts clean
    assert cstr.lib().is_check_build
    assert cstr.cstr_debug_bounds_status(reset=False) == (0, 0, 0, 0)


@pytest.mark.parametrize("seed", range(12))
def test_table_random_small(checked, seed):
    table_cases.test_random_small(seed)


def test_table_degenerate_cases(checked):
    table_cases.test_degenerate_cases()


@pytest.mark.parametrize("S", [4, 16, 17, 64, 65])
def test_table_small_automaton_kernels(checked, S):
    table_cases.test_small_automaton_kernels(S)


@pytest.mark.parametrize("case", ["string", "one_class", "eos_and_terminals"])
def test_table_duplicate_column_pass(checked, case):
    table_cases.test_few_byte_classes_take_the_duplicate_column_pass(case)


@pytest.mark.parametrize("case", ["plain", "eos", "terminals", "dense_walker"])
def test_table_sparse_automata(checked, case):
    table_cases.test_sparse_automata_are_renumbered_and_pruned(case)


def test_table_long_prefixes_rebuild_and_download(checked):
    table_cases.test_long_shared_prefixes_and_long_suffixes()
    table_cases.test_rebuild_reuses_the_table_and_wide_capacity()
    table_cases.test_download_slabs_of_any_alignment()


def test_table_staged_rows_path(checked):
    # 9,300 states with 256 byte classes: the bulk-copy builder (one CTA over all states)
    import numpy as np
    from synth import random_range_dfa
    rng = np.random.default_rng(3)
    dfa = random_range_dfa(9300, seed=4)
    vb, vo = table_cases.random_vocab(rng, 900, max_len=12)
    (table,) = table_cases.gpu_tables([dfa], vb, vo, eos_id=5)
    table_cases.check_table(table, dfa, vb, vo, eos_id=5,
                            states=[0, 1, 15, 16, 511, 512, 4000, 9215, 9216, 9298, 9299])


@pytest.mark.parametrize("seed", range(16))
def test_step_random_small(checked, seed):
    step_cases.test_random_small(seed)


def test_step_edge_cases(checked):
    step_cases.test_ties_signed_zero_nan_inf_across_chunks()
    step_cases.test_inactive_bad_and_empty_rows()
    step_cases.test_eos_token()
    step_cases.test_mixed_tables_and_bad_table_index()
    step_cases.test_many_rows_small_vocabulary()


def test_step_workloads(checked):
    step_cases.decode_and_check("api_1k", pool=4)
    step_cases.decode_and_check("json_32k", steps=24, pool=2)


@pytest.mark.parametrize("seed", range(4))
def test_terminals_random_small(checked, seed):
    term_cases.test_random_small(seed)


def test_speculative(checked):
    spec_cases.test_accept_draft_random()
    spec_cases.test_speculative_loop_matches_oracle()


@pytest.mark.parametrize("seed", range(4))
def test_pda_random(checked, seed):
    pda_cases.test_random_pdas_table_and_decode_loop(seed)


def test_pda_tables_and_loops(checked):
    pda_cases.test_table_anbn_figure5_vocabulary()
    pda_cases.test_table_dyck_and_eos()
    pda_cases.test_decode_loop_anbn_deep_pops()
    pda_cases.test_inactive_rows_bad_stacks_and_overflow()
