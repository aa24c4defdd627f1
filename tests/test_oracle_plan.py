"""Pins for the oracle's cache state machine and miss split (CPU only)."""
import os
from collections import OrderedDict
from fractions import Fraction

import numpy as np
import pytest

from oracle import ftmoe_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def _table1():
    out = {}
    for ln in _rows("table1_bandwidths.txt"):
        name, bp, bh = ln.split()
        out[name] = (int(round(float(bp) * 1000)), int(round(float(bh) * 1000)))   # MB/s
    return out


def cm_for(S=1 << 20, bf=50000, br=0, bz=50000, bh=6000000, R=1, Tz=64, Tg=128):
    return O.CostModel(expert_bytes=S, bw_fill=bf, bw_zc_residual=br, bw_zc=bz, bw_hbm=bh,
                       reuse_credit=R, zc_tokens_per_pass=Tz, hbm_tokens_per_pass=Tg)


# ---- q*: the paper's printed example and Table 1 ---------------------------------------

def test_fig2_worked_split():
    routed, hits, m, fills, inplace = map(int, _rows("fig2_miss_split.txt")[0].split())
    assert routed - hits == m and fills + inplace == m
    t1 = _table1()
    for system in ("4060-laptop", "PRO-6000"):
        bp, bh = t1[system]
        assert O.fill_count_bw(m, bp, bh - bp) == fills


def test_q_is_rounded_m_bp_over_bh_on_table1():
    for bp, bh in _table1().values():
        for m in range(0, 40):
            exact = Fraction(m * bp, bh)                      # Eq. 4
            rounded = int(exact + Fraction(1, 2))             # half up
            want = 0 if m == 0 else max(1, rounded)           # at least one miss is always filled (Eq. 4)
            assert O.fill_count_bw(m, bp, bh - bp) == want


def test_q_degenerates_to_pure_fill_without_residual():
    for m in range(0, 50):
        assert O.fill_count_bw(m, 52700, 0) == m            # B_Host -> B_PCIe  =>  q* -> m


# ---- hand-worked trace -----------------------------------------------------------------

def _parse_trace():
    steps = []
    for ln in _rows("lru_trace.txt"):
        routed, H, F, Z, table = [p.strip() for p in ln.split("|")]
        counts = {int(a.split(":")[0]): int(a.split(":")[1]) for a in routed.split()}
        H = [] if H == "-" else [int(v) for v in H.split()]
        Z = [] if Z == "-" else [int(v) for v in Z.split()]
        fills = []
        if F != "-":
            for item in F.split():
                e, rest = item.split(">")
                s, ev = rest.rstrip(")").split("(")
                fills.append((int(e), int(s), int(ev)))
        steps.append((counts, H, fills, Z, [int(v) for v in table.split()]))
    return steps


def test_hand_worked_trace():
    st = O.CacheState(6, 3)
    cm = cm_for()
    for t, (counts, H, fills, Z, table) in enumerate(_parse_trace()):
        count = np.zeros(6, dtype=np.int32)
        for e, n in counts.items():
            count[e] = n
        p = O.plan(st, count, cm)
        assert p.step == t
        assert p.hit == H
        assert [(e, s, ev) for e, s, ev in zip(p.fill_order, p.fill_slot, p.fill_evicted)] == fills
        assert p.zc == Z
        assert st.slot_expert.tolist() == table


# ---- classical LRU reduction -----------------------------------------------------------

def _lru_hits(trace, n_slots):
    lru = OrderedDict()
    hits = 0
    for e in trace:
        if e in lru:
            hits += 1
            lru.move_to_end(e)
        else:
            if n_slots == 0:
                continue
            if len(lru) >= n_slots:
                lru.popitem(last=False)
            lru[e] = True
    return hits


def test_single_token_single_choice_is_textbook_lru():
    rng = np.random.default_rng(3)
    E = 12
    trace = rng.zipf(1.5, size=600) % E
    prev = -1
    for n_slots in range(0, E + 1):
        st = O.CacheState(E, n_slots)
        hits = 0
        for e in trace:
            count = np.zeros(E, dtype=np.int32)
            count[e] = 1
            p = O.plan(st, count, cm_for())
            hits += len(p.hit)
        assert hits == _lru_hits(trace, n_slots)
        assert hits >= prev            # inclusion property of LRU
        prev = hits


# ---- closed forms ----------------------------------------------------------------------

def _random_counts(rng, E, T, k):
    ids = np.stack([rng.choice(E, size=k, replace=False) for _ in range(T)])
    return np.bincount(ids.reshape(-1), minlength=E).astype(np.int32)


def test_full_cache_has_only_compulsory_misses():
    rng = np.random.default_rng(4)
    E = 16
    st = O.CacheState(E, E)
    seen = set()
    fills = 0
    for step in range(60):
        count = _random_counts(rng, E, 3, 2)
        p = O.plan(st, count, cm_for())
        assert p.zc == [] and all(ev == -1 for ev in p.fill_evicted)
        assert set(p.miss) == set(p.routed) - seen
        seen |= set(p.routed)
        fills += len(p.fill)
    assert fills == len(seen)
    # warm pass over everything, then zero misses for ever ("zero misses at 100% cache")
    O.plan(st, np.ones(E, dtype=np.int32), cm_for())
    for step in range(20):
        p = O.plan(st, _random_counts(rng, E, 3, 2), cm_for())
        assert p.miss == []


def test_no_slots_means_everything_in_place():
    rng = np.random.default_rng(5)
    st = O.CacheState(8, 0)
    for _ in range(5):
        count = _random_counts(rng, 8, 4, 2)
        p = O.plan(st, count, cm_for())
        assert p.hit == [] and p.fill == [] and p.zc == p.routed
        assert all(p.loc[e] == O.LOC_ZERO_COPY for e in p.routed)


def test_empty_step_does_not_advance():
    st = O.CacheState(8, 4)
    assert O.plan(st, np.zeros(8, dtype=np.int32), cm_for()) is None
    assert st.step == 0


def test_myopic_mode_fills_only_multi_pass_experts():
    # R = 0 and B_z == B_f: a fill only pays when the in-place branch needs several link passes
    cm = cm_for(R=0, Tz=4, Tg=128)
    st = O.CacheState(8, 8)
    count = np.array([1, 4, 5, 9, 0, 0, 0, 0], dtype=np.int32)
    p = O.plan(st, count, cm)
    assert p.fill == [2, 3] and p.zc == [0, 1]
    assert p.fill_order == [3, 2]


# ---- invariants + an independent naive implementation -----------------------------------

class NaivePlan:
    """A second statement of the same rules with different data structures (dict per expert)."""

    def __init__(self, E, n_slots):
        self.res = {}                       # expert -> [slot, stamp]
        self.free = list(range(n_slots))
        self.t = 0

    def step(self, count, cm):
        t = self.t
        U = [e for e in range(len(count)) if count[e] > 0]
        H = [e for e in U if e in self.res]
        M = [e for e in U if e not in self.res]
        for e in H:
            self.res[e][1] = t
        old = sorted((st, e) for e, (s, st) in self.res.items() if st < t)
        cand = [(s, -1) for s in sorted(self.free)] + [(self.res[e][0], e) for st, e in old]
        S = cm.expert_bytes
        tz, tf, th = S * 1000 // cm.bw_zc, S * 1000 // cm.bw_fill, S * 1000 // cm.bw_hbm
        elig = []
        for e in M:
            n = int(count[e])
            gain = ((n + cm.zc_tokens_per_pass - 1) // cm.zc_tokens_per_pass) * tz \
                - tf - ((n + cm.hbm_tokens_per_pass - 1) // cm.hbm_tokens_per_pass) * th \
                + cm.reuse_credit * (tz - th)
            if gain > 0:
                elig.append((-n, e))
        elig.sort()
        m = len(M)
        if m == 0:
            qbw = 0
        else:
            qbw = max(1, int(Fraction(m * cm.bw_fill, cm.bw_fill + cm.bw_zc_residual) + Fraction(1, 2)))
        q = min(qbw, len(elig), len(cand))
        F = [e for _, e in elig[:q]]
        slots, evicted = [], []
        for e, (s, ev) in zip(F, cand):
            if ev >= 0:
                del self.res[ev]
            else:
                self.free.remove(s)
            self.res[e] = [s, t]
            slots.append(s)
            evicted.append(ev)
        self.t += 1
        return H, M, F, slots, evicted, [e for e in M if e not in F]


@pytest.mark.parametrize("n_slots,br,R,Tz", [(4, 0, 1, 64), (5, 35700, 1, 64), (3, 24600, 0, 2), (16, 4800, 1, 64)])
def test_invariants_and_naive_agree(n_slots, br, R, Tz):
    rng = np.random.default_rng(n_slots * 7 + R)
    E = 16
    bf = 11800 if br == 35700 else 52700
    cm = cm_for(bf=bf, br=br, bz=bf, R=R, Tz=Tz)     # B_z == B_f: with R >= 1 every miss is eligible
    st = O.CacheState(E, n_slots)
    nv = NaivePlan(E, n_slots)
    prev_stamp = st.slot_stamp.copy()
    for step in range(120):
        T = int(rng.integers(1, 7))
        count = _random_counts(rng, E, T, 3)
        before_expert = st.slot_expert.copy()
        p = O.plan(st, count, cm)
        H, M, F, slots, evicted, Z = nv.step(count, cm)
        assert (p.hit, p.miss, p.fill_order, p.fill_slot, p.fill_evicted, p.zc) == (H, M, F, slots, evicted, Z)
        # partition
        assert sorted(p.hit + p.fill + p.zc) == p.routed
        assert not (set(p.hit) & set(p.fill)) and not (set(p.fill) & set(p.zc))
        # tables mutually inverse, no expert twice
        occ = [int(e) for e in st.slot_expert if e >= 0]
        assert len(occ) == len(set(occ))
        for s, e in enumerate(st.slot_expert):
            if e >= 0:
                assert st.expert_slot[e] == s
        for e, s in enumerate(st.expert_slot):
            if s >= 0:
                assert st.slot_expert[s] == e
        # hits are never evicted; in-place experts leave residency unchanged
        assert not (set(p.fill_evicted) & set(p.hit))
        for e in p.zc:
            assert st.expert_slot[e] == -1
        untouched = set(range(n_slots)) - set(p.fill_slot)
        for s in untouched:
            assert st.slot_expert[s] == before_expert[s]
        # stamps
        assert np.all(st.slot_stamp <= p.step) and np.all(st.slot_stamp >= prev_stamp)
        prev_stamp = st.slot_stamp.copy()
        # at least one fill whenever something is eligible and a slot can be had
        evictable = sum(1 for s in range(n_slots) if before_expert[s] < 0 or before_expert[s] not in p.hit)
        if p.miss and evictable and R >= 1:
            assert len(p.fill) >= 1
        # loc
        for e in range(E):
            if e in p.hit or e in p.fill:
                assert p.loc[e] == st.expert_slot[e] >= 0
            elif e in p.zc:
                assert p.loc[e] == O.LOC_ZERO_COPY
            else:
                assert p.loc[e] == O.LOC_NOT_ROUTED
