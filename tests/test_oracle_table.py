"""The oracle's chunk-swap table update against a hand-worked trace and an independent set model (CPU only)."""
import os

import numpy as np
import pytest
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


# ------------------------------------------------------------------ overlapping chunks, permanent base, lag-delta release
def _parse_lag_trace():
    rows = []
    for line in open(os.path.join(os.path.dirname(GOLDEN), "lag_update_trace.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        step, chunk, table, stamps, fetched, released, hits = [x.strip() for x in line.split("|")]
        rows.append(dict(step=int(step), chunk=int(chunk), table=[int(x) for x in table.split()],
                         stamps=[None if x == "x" else int(x) for x in stamps.split()],
                         fetched=[] if fetched == "-" else [tuple(int(y) for y in x.split("->")) for x in fetched.split()],
                         released=[] if released == "-" else [int(x) for x in released.split()], hits=int(hits)))
    return rows


def test_lag_update_follows_the_hand_worked_trace():
    """Dynamic Chunk Selection with a permanent prefill base and lag-delta release, against a trace worked by hand."""
    tab = np.array([0, 4, -1, -1, -1, -1], np.int32)
    stamp = np.array([-1, -2, 0, 0, 0, 0], np.int64)
    for row in _parse_lag_trace():
        segs = [row["chunk"], row["chunk"] + 1]
        plan, released, hits = wo.lag_update(tab, stamp, 2, segs, row["step"], 2)
        assert tab.tolist() == row["table"], row
        assert plan == row["fetched"], row
        assert sorted(released) == sorted(row["released"]), row
        assert hits == row["hits"], row
        for j, want in enumerate(row["stamps"]):
            if want is not None:
                assert stamp[2 + j] == want, row


def test_select_segments_overlapping_chunks_against_brute_force():
    """Chunk j = segments j, j+1 ranked by the mean over its tokens (float32), ties to the lower chunk; the segment list
    is the chunks' segments in rank order without repeats."""
    rng = np.random.default_rng(5)
    for trial in range(200):
        n_seg = int(rng.integers(1, 12))
        k = int(rng.integers(1, 5))
        sums = rng.random(n_seg).astype(np.float32)
        if trial % 5 == 0:
            sums[:] = np.float32(0.25)          # all ties
        lens = np.full(n_seg, 25, np.int32)
        lens[-1] = int(rng.integers(1, 26))     # ragged last segment
        ch, sg = wo.select_segments(sums, lens, k)
        n_ch = n_seg - 1 if n_seg > 1 else 1
        keys = [(np.float32(sums[j] + sums[j + 1]) / np.float32(lens[j] + lens[j + 1])) if n_seg > 1 else sums[0] / np.float32(lens[0])
                for j in range(n_ch)]
        order = sorted(range(n_ch), key=lambda j: (-float(keys[j]), j))[:min(k, n_ch)]
        assert ch.tolist() == order
        want = []
        for j in order:
            for g in ((j, j + 1) if n_seg > 1 else (j,)):
                if g not in want:
                    want.append(g)
        assert sg.tolist() == want


@pytest.mark.parametrize("delta", [0, 1, 3])
def test_lag_update_equals_the_window_set_model(delta):
    """Independent model: after step s the dynamic set is exactly the union of the segments selected in the last
    max(delta, 1) steps, minus the base; the plan is what was selected now and was not resident before; the pool of
    2*k*(delta+1) dynamic slots never overflows; base slots never change."""
    rng = np.random.default_rng(11 + delta)
    n_seg, k, s_base = 40, 3, 8
    D = 2 * k * (delta + 1)
    base = rng.choice(n_seg, s_base, replace=False).astype(np.int32)
    tab = np.concatenate([base, np.full(D, -1, np.int32)]).astype(np.int32)
    stamp = np.zeros(s_base + D, np.int64)
    history = []
    for step in range(60):
        chunks = rng.choice(n_seg - 1, k, replace=False) if step % 7 else np.array([3, 4, 5])   # overlapping chunks too
        segs = []
        for j in chunks:
            for g in (int(j), int(j) + 1):
                if g not in segs:
                    segs.append(g)
        before = set(int(x) for x in tab if x >= 0)
        plan, released, hits = wo.lag_update(tab, stamp, s_base, segs, step, delta)
        history.append(set(segs))
        window = set().union(*history[-max(delta, 1):]) - set(base.tolist())
        assert set(int(x) for x in tab[s_base:] if x >= 0) == window
        assert tab[:s_base].tolist() == base.tolist()
        assert [g for g, _ in plan] == [g for g in segs if g not in before]
        assert hits == len([g for g in segs if g in before])
        assert set(released) == (before - set(base.tolist())) - window
        assert len(set(int(x) for x in tab if x >= 0)) == int((tab >= 0).sum())     # no segment twice
