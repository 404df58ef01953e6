"""Closed-loop decode simulation harness (inputs and bookkeeping only).

The paper's simulated verifier (Section 4.1, "Simulated Ablations"): with a
known ground-truth response, greedy speculative verification accepts a drafted
token exactly when it equals the ground-truth token at its position.  For a
draft TREE that is the unique root-to-node path spelling a prefix of the truth
(siblings carry distinct tokens).  Each step then appends the accepted tokens
plus one bonus token; a finished request's output goes into the global tree
and its slot is refilled with a fresh request.
"""
from __future__ import annotations

from typing import Dict, List

import numpy as np

from .generator import Workload


def accept_longest_path(tokens: np.ndarray, parents: np.ndarray, n: int, truth: np.ndarray) -> int:
    """Number of draft tokens accepted against `truth` (the tokens that really follow)."""
    cur, depth = -1, 0
    while depth < len(truth):
        nxt = -1
        for j in range(n):
            if parents[j] == cur and tokens[j] == truth[depth]:
                nxt = j
                break
        if nxt < 0:
            break
        cur, depth = nxt, depth + 1
    return depth


class ClosedLoop:
    """Tracks, for every slot, the current request, its hidden continuation and a cursor."""

    def __init__(self, w: Workload, n_slots: int, prompt_len: int = None, out_lo: int = None, out_hi: int = None):
        self.w, self.n_slots = w, n_slots
        self.prompt_len = w.cfg.prompt_len if prompt_len is None else prompt_len
        self.out_lo = w.cfg.out_len_lo if out_lo is None else out_lo
        self.out_hi = w.cfg.out_len_hi if out_hi is None else out_hi
        self.next_request = 0
        self.request = [0] * n_slots
        self.prompt: List[np.ndarray] = [None] * n_slots
        self.truth: List[np.ndarray] = [None] * n_slots
        self.cursor = [0] * n_slots
        self.accepted_total = 0
        self.drafted_total = 0
        self.slot_steps = 0
        self.finished = 0

    def _new_request(self, slot: int) -> np.ndarray:
        r = self.next_request
        self.next_request += 1
        self.request[slot] = r
        self.prompt[slot] = self.w.prompt(r, length=self.prompt_len)
        span = self.out_hi - self.out_lo + 1
        out_len = self.out_lo + (self.w.output_length(r) - self.w.cfg.out_len_lo) % span
        self.truth[slot] = self.w.continuation(r, self.prompt[slot], length=out_len)
        self.cursor[slot] = 0
        return self.prompt[slot]

    def start(self):
        """Append items that load a fresh request into every slot: (slots, token lists, reset flags)."""
        return list(range(self.n_slots)), [self._new_request(s) for s in range(self.n_slots)], [1] * self.n_slots

    def advance(self, out: Dict[str, np.ndarray]):
        """Consume one step's drafts (row i belongs to slot i).  Returns the append items of
        this step: accepted + bonus tokens per slot, then for every request that finished a
        global insert of its output (slot -1) and the refill of its slot."""
        slots, lists, reset = [], [], []
        after_slots, after_lists, after_reset = [], [], []
        for s in range(self.n_slots):
            truth, cur = self.truth[s], self.cursor[s]
            n = int(out["n_draft"][s])
            acc = accept_longest_path(out["tokens"][s], out["parents"][s], n, truth[cur:])
            take = min(acc + 1, len(truth) - cur)                 # accepted drafts + one bonus token
            self.accepted_total += acc
            self.drafted_total += n
            self.slot_steps += 1
            new = truth[cur:cur + take]
            self.cursor[s] = cur + take
            if self.cursor[s] >= len(truth):
                self.finished += 1
                after_slots.append(-1); after_lists.append(truth.copy()); after_reset.append(0)
                after_slots.append(s); after_lists.append(self._new_request(s)); after_reset.append(1)
            else:
                slots.append(s); lists.append(new); reset.append(0)
        return slots + after_slots, lists + after_lists, reset + after_reset

    def summary(self) -> dict:
        steps = max(self.slot_steps, 1)
        return {"mean_accepted_drafts": self.accepted_total / steps,
                "mean_accepted_tokens_incl_bonus": self.accepted_total / steps + 1.0,
                "acceptance_rate": self.accepted_total / max(self.drafted_total, 1),
                "finished_requests": self.finished}
