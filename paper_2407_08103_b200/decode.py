"""Batched constrained decoding driver over the libcstr binding.

Holds the per-batch device state (one automaton state per row, Algorithm 2's
``q``) and the step workspace; every step is one ``cstr_step`` call.  The LM
that produces the logits is outside this package.
"""

from __future__ import annotations

import torch

from . import cstr


class ConstrainedDecoder:
    """``tables``: one built Table, or several for a mixed-constraint batch with
    ``row_table`` (int32 per row) choosing each row's table."""

    def __init__(self, tables, batch: int, row_table=None, device="cuda:0"):
        self.tables = [tables] if isinstance(tables, cstr.Table) else list(tables)
        self.batch = batch
        self.device = torch.device(device)
        self.infos = [cstr.cstr_table_info(t) for t in self.tables]
        self.vocab_size = self.infos[0]["vocab_size"]
        self.ws = cstr.cstr_workspace_create(batch)
        self.row_table = None
        if row_table is not None:
            self.row_table = torch.as_tensor(row_table, dtype=torch.int32).to(self.device)
        self.states = torch.empty(batch, dtype=torch.int32, device=self.device)
        self.tokens = torch.empty(batch, dtype=torch.int32, device=self.device)
        self.accept = torch.empty(batch, dtype=torch.uint8, device=self.device)
        self._start = self._start_states()
        self.reset()

    def _start_states(self):
        starts = torch.tensor([i["start_state"] for i in self.infos], dtype=torch.int32,
                              device=self.device)
        if self.row_table is None:
            return starts[0].expand(self.batch).contiguous()
        return starts[self.row_table.long()].contiguous()

    def reset(self):
        """All rows back to their automaton's start state (Algorithm 2: q <- I)."""
        self.states.copy_(self._start)

    def step(self, logits, noise=None, masked_out=None, stream=None):
        """One decoding step; returns ``(tokens, masked_logits)`` (device tensors;
        ``tokens`` is reused by the next call)."""
        if masked_out is None:
            masked_out = torch.empty_like(logits)
        cstr.cstr_step(self.tables, logits, self.states, self.tokens, masked_out, self.ws,
                       noise=noise, row_table=self.row_table, accept_out=self.accept,
                       stream=stream)
        return self.tokens, masked_out

    def status(self, stream=None):
        """(rows with an out-of-range state, active rows without any allowed token) since last call."""
        return cstr.cstr_step_status(self.ws, stream)


class PushdownDecoder:
    """Per-batch state of Algorithm 3: one PDA state, one stack (``stack_cap``
    symbols) and its depth per row; every step is one ``cstr_pda_step`` call."""

    def __init__(self, table, batch: int, stack_cap: int = 64, device="cuda:0"):
        self.table = table
        self.batch = batch
        self.device = torch.device(device)
        self.info = cstr.cstr_pda_table_info(table)
        self.vocab_size = self.info["vocab_size"]
        self.ws = cstr.cstr_pda_workspace_create(table, batch)
        self.states = torch.empty(batch, dtype=torch.int32, device=self.device)
        self.stacks = torch.zeros((batch, stack_cap), dtype=torch.int32, device=self.device)
        self.depths = torch.empty(batch, dtype=torch.int32, device=self.device)
        self.tokens = torch.empty(batch, dtype=torch.int32, device=self.device)
        self.accept = torch.empty(batch, dtype=torch.uint8, device=self.device)
        self.reset()

    def reset(self):
        """All rows back to the start state with an empty stack (Algorithm 3: q <- I, s <- empty)."""
        self.states.fill_(self.info["start_state"])
        self.depths.zero_()

    def restart_finished(self):
        """Replace every finished row (state -1) by a fresh sequence."""
        done = self.states < 0
        self.states.masked_fill_(done, self.info["start_state"])
        self.depths.masked_fill_(done, 0)

    def step(self, logits, noise=None, masked_out=None, stream=None):
        if masked_out is None:
            masked_out = torch.empty_like(logits)
        cstr.cstr_pda_step(self.table, logits, self.states, self.stacks, self.depths, self.tokens,
                           masked_out, self.ws, noise=noise, accept_out=self.accept, stream=stream)
        return self.tokens, masked_out

    def status(self, stream=None):
        """(inactive rows other than finished ones, rows without an allowed token,
        rows whose stack outgrew ``stack_cap``) since the last call."""
        return cstr.cstr_pda_step_status(self.ws, stream)
