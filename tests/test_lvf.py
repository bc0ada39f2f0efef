"""The list maker that follows the paper's scheduler (section 4.2): Virtual Lag Time and one
Largest-VLT-First decision (Algorithm 1), pinned by hand-worked values, and the lists the toy replay
makes from them checked for validity with the oracle's own list check and tag model."""
import numpy as np
import pytest

from oracle.kv_definition import TagModel, check_lists
from paper_2601_20309_b200 import workload as W

P = W.LVFParams()          # the paper's evaluation settings: alpha 3, beta_B 0, beta_F 0.5, SLOs 5 s / 100 ms


def test_paper_settings():
    assert (P.alpha, P.beta_b, P.beta_f, P.slo_first_s, P.slo_between_s, P.b_xfer) == (3.0, 0.0, 0.5, 5.0, 0.1, 2400)


def test_vlt_of_a_waiting_request_is_zero_within_tolerance_then_grows_with_the_wait():
    # tolerance = beta_F * S_F = 0.5 * 5 s = 2.5 s after arrival
    assert W.vlt("waiting", 12.0, 10.0, P) == 0.0             # 2.0 s waited
    assert W.vlt("waiting", 12.5, 10.0, P) == 0.0             # exactly at the tolerance
    assert W.vlt("waiting", 14.0, 10.0, P) == pytest.approx(1.5)
    assert W.vlt("waiting", 14.0, 10.0, W.LVFParams(beta_f=0.0)) == pytest.approx(4.0)


def test_vlt_of_a_rotary_request_is_weighted_by_alpha():
    # beta_B = 0: lag counts from the last token; alpha = 3
    assert W.vlt("rotary", 7.25, 7.0, P) == pytest.approx(0.75)
    assert W.vlt("rotary", 7.0, 7.0, P) == 0.0
    q = W.LVFParams(alpha=2.0, beta_b=1.0)                    # tolerance = 1 * 100 ms
    assert W.vlt("rotary", 7.05, 7.0, q) == 0.0
    assert W.vlt("rotary", 7.25, 7.0, q) == pytest.approx(2.0 * 0.15)
    q = W.LVFParams(beta_b=-1.0)                              # a negative tolerance: lag before any time has passed
    assert W.vlt("rotary", 7.0, 7.0, q) == pytest.approx(3.0 * 0.1)


def test_vlt_of_a_running_request_is_negative_and_falls_as_it_runs():
    assert W.vlt("running", 9.4, 8.0, P) == pytest.approx(-1.4)
    assert W.vlt("running", 8.0, 8.0, P) == 0.0
    assert W.vlt("running", 9.4, 8.0, W.LVFParams(alpha=10.0, beta_b=3.0, beta_f=3.0)) == pytest.approx(-1.4)
    with pytest.raises(ValueError):
        W.vlt("finished", 1.0, 0.0, P)


# running A (10 blocks, has run 3 s), running B (6 blocks, 1 s), waiting C (8 blocks, VLT 2.0), rotary D (5 blocks, 0.9)
FOUR = [(1, "running", -3.0, 10), (2, "running", -1.0, 6), (3, "waiting", 2.0, 8), (4, "rotary", 0.9, 5)]


def test_lvf_worked_example_wide_budget():
    # 2 free blocks, budget 12: sorted C, D, B, A; 14 blocks to give: C (8) -> 6 left, D (5) -> 1 left;
    # B_swap = 12 - 1 = 11 = the 13 blocks of C and D minus the 2 free ones; from the tail: A frees 10 (1 still
    # missing), so B goes too
    assert W.lvf_select(FOUR, b_hbm=2, b_xfer=12) == ([1, 2], [3, 4])


def test_lvf_worked_example_tight_budget():
    # budget 4: 6 blocks to give: C (8) does not fit, D (5) does -> 1 left; B_swap = 4 - 1 = 3; A alone frees enough
    assert W.lvf_select(FOUR, b_hbm=2, b_xfer=4) == ([1], [4])
    # nothing fits: no one is prioritized and B_swap = 0 - 0... budget 0 with 2 free blocks: nobody preempted
    assert W.lvf_select(FOUR, b_hbm=2, b_xfer=0) == ([], [])


def test_lvf_without_contention_falls_back_to_first_come_first_served():
    assert W.lvf_select(FOUR, b_hbm=13, b_xfer=12) == ([], [3, 4])        # C and D need 13 blocks: they fit
    assert W.lvf_select(FOUR, b_hbm=12, b_xfer=12) == ([1], [3, 4])       # one block short: one preemption
    assert W.lvf_select([r for r in FOUR if r[1] == "running"], b_hbm=0, b_xfer=100) == ([], [])


def test_lvf_takes_the_most_lagging_first_and_preempts_the_longest_running_first():
    reqs = [(1, "running", -0.5, 4), (2, "running", -9.0, 4), (3, "running", -2.0, 4),
            (10, "waiting", 0.0, 4), (11, "rotary", 6.0, 4), (12, "waiting", 3.0, 4), (13, "rotary", 0.0, 4)]
    # no free blocks, budget 8: two of the four idle requests fit: the rotary one with VLT 6, then the waiting one
    # with VLT 3; 8 blocks must be freed: the request that has run 9 s, then the one that has run 2 s
    assert W.lvf_select(reqs, b_hbm=0, b_xfer=8) == ([2, 3], [11, 12])
    # equal VLTs keep the given order: with room for three, request 10 (listed before 13) is the third
    assert W.lvf_select(reqs, b_hbm=0, b_xfer=12) == ([2, 3, 1], [11, 12, 10])
    # a running request whose VLT is still 0 (it started this very step) is neither prioritized nor preempted
    reqs2 = [(1, "running", 0.0, 4), (2, "running", -1.0, 4), (10, "waiting", 5.0, 8)]
    assert W.lvf_select(reqs2, b_hbm=0, b_xfer=8) == ([2], [10])


@pytest.fixture(scope="module")
def lvf_small():
    return W.config5_lvf(rate=3.0, n_steps=500, shape=W.KVShape(2, 16, 2, 64), duration_s=30.0, max_tokens=1024,
                         params=W.LVFParams(b_xfer=40))


def test_lvf_replay_emits_valid_rotations(lvf_small):
    w = lvf_small
    assert len(w.steps) == 500
    both = sum(1 for s in w.steps if s.n_out and s.n_in)
    assert both > 20 and w.extra["preempted"].sum() > 20 and w.extra["resumed"].sum() > 20
    tags = TagModel(w.nb_gpu, w.nb_host)
    for s in w.steps:
        a = (s.out_gpu.tolist(), s.out_host.tolist(), s.in_host.tolist(), s.in_gpu.tolist())
        assert check_lists(w.nb_gpu, w.nb_host, *a) == 0                  # the oracle's own validation, no overlap allowed
        assert tags.rotate(*a) == 0
    w.table.check_consistent()


def test_lvf_replay_obeys_the_decision_it_is_built_on(lvf_small):
    """Swap-outs per step are bounded by what Algorithm 1 can ask for (B_swap <= B_xfer, plus the request
    that crosses the line), and a step never brings in more than was free."""
    w = lvf_small
    longest = -(-1024 * 2 // 16)                                          # prompt + output, both clipped at 1024 tokens
    assert max(s.n_out for s in w.steps) <= 40 + longest
    assert max(s.n_in for s in w.steps) <= w.nb_gpu
    assert w.extra["admitted"].sum() <= w.extra["arrivals"]


def test_lvf_replay_is_seeded():
    a = W.config5_lvf(rate=3.0, n_steps=120, shape=W.KVShape(2, 16, 2, 64), duration_s=8.0, max_tokens=512)
    b = W.config5_lvf(rate=3.0, n_steps=120, shape=W.KVShape(2, 16, 2, 64), duration_s=8.0, max_tokens=512)
    for x, y in zip(a.steps, b.steps):
        assert np.array_equal(x.out_gpu, y.out_gpu) and np.array_equal(x.in_host, y.in_host)
