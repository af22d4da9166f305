"""The transition estimate, the admission gate (Eq. 2) and the horizon H_x, against the plain restatement in
oracle/admission.py and against what the paper says about them in words (Section 4.3)."""
import math

import pytest
from hypothesis import given, settings, strategies as st

from oracle import admission as A
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I


def test_gate_statements_of_the_paper():
    # the ratio counts the steps until the savings have paid for the move: 12 s of transition against 1.5 s saved per step pays back in 8 steps
    ok, pb = B.admit(12.0, 10.0, 8.5, gamma=0.5, h_x=16.0)
    assert pb == pytest.approx(8.0) and ok                      # 8 <= 0.5 * 16
    ok, _ = B.admit(12.0, 10.0, 8.5, gamma=0.5, h_x=15.9)
    assert not ok                                               # 8 > 7.95
    # no savings, no admission, whatever the horizon
    ok, pb = B.admit(0.001, 10.0, 10.0, gamma=1.0, h_x=1e9)
    assert not ok and math.isinf(pb)
    ok, _ = B.admit(0.001, 10.0, 11.0, gamma=1.0, h_x=1e9)
    assert not ok
    # with gamma = 0 nothing but the urgent path gets through, not even a free transition
    assert not B.admit(0.0, 10.0, 5.0, gamma=0.0, h_x=100.0)[0]
    assert B.admit(1e6, 10.0, 12.0, gamma=0.0, h_x=0.0, urgent=True)[0]       # urgent waives profitability
    # the paper's 1,000-step run: six transitions, 49.5 s in all; a transition of 49.5/6 s that saves 1 s per
    # step pays back in 8.25 steps
    ok, pb = B.admit(49.5 / 6, 62.353, 61.353, gamma=0.5, h_x=20)
    assert pb == pytest.approx(8.25) and ok
    with pytest.raises(B.NereusError):
        B.admit(1.0, 2.0, 1.0, gamma=1.5)
    with pytest.raises(B.NereusError):
        B.admit(-1.0, 2.0, 1.0)


@settings(max_examples=300, deadline=None)
@given(st.floats(0, 1e4), st.floats(0.01, 1e3), st.floats(0.01, 1e3), st.floats(0, 1), st.floats(0, 1e4),
       st.booleans())
def test_gate_matches_restatement(l_tran, cur, new, gamma, h_x, urgent):
    got, pb = B.admit(l_tran, cur, new, gamma, h_x, urgent)
    assert got == A.admit(l_tran, cur, new, gamma, h_x, urgent)
    want_pb = A.payback_steps(l_tran, cur, new)
    assert (math.isinf(pb) and math.isinf(want_pb)) or pb == pytest.approx(want_pb)
    if got and not urgent:                         # monotone: a larger margin or horizon never un-admits
        assert B.admit(l_tran, cur, new, min(1.0, gamma * 1.5), h_x * 2)[0]


def test_horizon():
    h = B.Horizon(0.5)
    assert h.h_steps == 1.0 and h.observed == 0                 # one step before the first interval
    assert h.crossing(40) == 40.0                               # the first observed interval replaces it
    assert h.crossing(20) == 30.0
    assert h.crossing(30) == 30.0
    ref = A.Horizon(0.25)
    lib = B.Horizon(0.25)
    for x in (7, 9, 100, 3, 3, 3):
        assert lib.crossing(x) == pytest.approx(ref.crossing(x))
    with pytest.raises(B.NereusError):
        B.Horizon(0.0)


def test_estimate_from_bytes():
    sh = I.LLAMA_8B
    d = B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.BF16)
    t = d.compile(B.Plan(1, 1), B.Plan(4, 2))
    rd, wr = t.bytes()
    assert t.estimate(6800.0, 5e-6) == pytest.approx(A.estimate_seconds(rd, wr, 6800.0, 5e-6))
    assert t.estimate(6800.0) == pytest.approx(32_124_239_872 / 6.8e12)
    back = d.compile(B.Plan(4, 2), B.Plan(1, 1))
    chain = B.Transition.fuse([t, back], chained=True)
    assert chain.estimate(6800.0) == pytest.approx(t.estimate(6800.0) + back.estimate(6800.0))
    k3 = d.compile_replicated(B.Plan(4, 2), B.Plan(4, 2), 3)
    r3, w3 = k3.bytes()
    assert w3 == 3 * r3 and k3.estimate(1000.0) == pytest.approx((r3 + w3) / 1e12)
    with pytest.raises(B.NereusError):
        t.estimate(0.0)
