"""The oracle's chunk-swap table update against a hand-worked trace and an independent set model (CPU only)."""
import os

import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import wnw_oracle as wo

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table_update_trace.txt")


def test_hand_worked_trace():
    rows = [l.strip() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    init = [x.strip() for x in rows[0].split("|")]
    slot = np.array(init[2].split(), np.int32); stamp = np.array(init[3].split(), np.int64)
    for row in rows[1:]:
        step, sel, want_slot, want_stamp, want_plan = [x.strip() for x in row.split("|")]
        plan, _ = wo.table_update(slot, stamp, [int(x) for x in sel.split()], int(step), 2)
        assert slot.tolist() == [int(x) for x in want_slot.split()], row
        assert stamp.tolist() == [int(x) for x in want_stamp.split()], row
        got = " ".join(f"{c}>{s}({e})" for c, s, e in plan) or "-"
        assert got == want_plan, row


class SetModel:
    """Independent restatement with dicts: residents map chunk -> (slot, last-selected time)."""

    def __init__(self, S, init):
        self.S = S
        self.where = {c: j for j, c in enumerate(init)}          # chunk -> slot
        self.when = {c: -1 - j for j, c in enumerate(init)}      # chunk -> recency

    def update(self, sel, step, k):
        recalled, evicted = [], []
        for r, c in enumerate(sel):
            now = step * k + (k - 1 - r)
            if c not in self.where:
                used = set(self.where.values())
                free = [j for j in range(self.S) if j not in used]
                if free:
                    j = free[0]
                else:
                    victim = min((x for x in self.where if x not in sel), key=lambda x: self.when[x])
                    j = self.where.pop(victim); self.when.pop(victim); evicted.append(victim)
                self.where[c] = j
                recalled.append((c, j))
            self.when[c] = now
        return recalled, evicted

    def table(self):
        t = [-1] * self.S
        for c, j in self.where.items():
            t[j] = c
        return t


@settings(max_examples=300, deadline=None)
@given(st.data())
def test_table_update_matches_set_model(data):
    C = data.draw(st.integers(3, 24))
    k = data.draw(st.integers(1, 3))
    S = data.draw(st.integers(k, C))
    n_init = data.draw(st.integers(0, S))
    init = data.draw(st.permutations(range(C)))[:n_init]
    slot = np.full(S, -1, np.int32); stamp = np.zeros(S, np.int64)
    slot[:n_init] = init; stamp[:n_init] = [-1 - j for j in range(n_init)]
    model = SetModel(S, list(init))
    last_stamp = stamp.copy()
    for step in range(data.draw(st.integers(1, 12))):
        sel = data.draw(st.permutations(range(C)))[:k]
        free_before = int((slot < 0).sum())
        plan, hits = wo.table_update(slot, stamp, sel, step, k)
        recalled, evicted = model.update(list(sel), step, k)
        assert slot.tolist() == model.table()
        assert [(c, j) for c, j, _ in plan] == recalled
        assert [e for _, _, e in plan if e >= 0] == evicted
        # invariants
        res = [c for c in slot.tolist() if c >= 0]
        assert len(res) == len(set(res)) <= S                       # partial permutation
        assert set(sel) <= set(res)                                 # every selected chunk resident afterwards
        assert hits + len(plan) == k
        assert len(evicted) == len(plan) - min(free_before, len(plan))
        changed = stamp != last_stamp
        assert (stamp[changed] > last_stamp[changed]).all()         # stamps only grow
        assert len(set(stamp[slot >= 0].tolist())) == len(res)      # and stay unique among residents
        last_stamp = stamp.copy()
