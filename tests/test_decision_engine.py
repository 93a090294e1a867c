"""PD decision engine: pins for the Python oracle, then the library's C functions against it (CPU only)."""
import math

import numpy as np
import pytest

from oracle import decision as od

FIELDS = ("B", "S", "r", "dL", "theta", "A", "b", "t_prefill", "T_over", "T_env", "K_bytes", "BW", "K_seq_bytes",
          "H_max_bytes", "prefill_tokens_per_worker")


def model(**kw):
    m = dict(B=64.0, S=10.0, r=200.0, dL=1000.0, theta=0.5, A=0.02, b=5e-4, t_prefill=1e-5, T_over=0.01, T_env=5.0,
             K_bytes=4096.0 * 36, BW=50e9, K_seq_bytes=32768 * 4096.0 * 36, H_max_bytes=400e9,
             prefill_tokens_per_worker=0.0)
    m.update(kw)
    return m


def c_model(m):
    import paper_2609_35158_b200 as pd

    return pd.pd_cost_model(*[float(m[f]) for f in FIELDS])


# ---------------------------------------------------------------- oracle pins

def test_eq1_special_cases():
    m = model(b=0.0, t_prefill=0.0)
    assert od.makespan_coloc(m, 7) == pytest.approx(10 * (200 * 0.02 + 0.01) + 5.0, rel=1e-15)
    m = model(A=0.0, T_over=0.0, T_env=0.0)
    # with no fixed costs the makespan is inversely proportional to the worker count
    assert od.makespan_coloc(m, 4) == pytest.approx(2 * od.makespan_coloc(m, 8), rel=1e-14)
    # hand evaluation: S [ (B dL / N) t_prefill + r (A + b B / N) + T_over ] + T_env
    assert od.makespan_coloc(model(), 8) == pytest.approx(10 * ((64 * 1000 / 8) * 1e-5 + 200 * (0.02 + 5e-4 * 8) + 0.01) + 5, rel=1e-15)


def test_eq2_eq3_special_cases_and_monotonicity():
    m = model(theta=0.0)
    t, tp, td = od.makespan_disagg(m, 3, 5)
    assert td == pytest.approx(10 * 200 * (0.02 + 5e-4 * 64 / 5), rel=1e-15)
    assert tp == pytest.approx(10 * ((64 * 1000 / 3) * 1e-5 + 64 * 1000 * 4096 * 36 / 50e9), rel=1e-15)
    assert t == max(tp, td) + 5.0
    # bubbles only add the fixed cost A (1 + theta): the KV term b B / N_D is unchanged
    t2, _, td2 = od.makespan_disagg(model(theta=1.0), 3, 5)
    assert td2 - td == pytest.approx(10 * 200 * 0.02 * 1.0, rel=1e-12)
    m = model()
    tds = [od.makespan_disagg(m, 1, nd)[2] for nd in range(1, 9)]
    tps = [od.makespan_disagg(m, n_p, 1)[1] for n_p in range(1, 9)]
    assert all(a > b for a, b in zip(tds, tds[1:])) and all(a > b for a, b in zip(tps, tps[1:]))
    # the transfer term lower-bounds the prefill path however many prefill workers there are
    assert od.makespan_disagg(m, 10 ** 9, 1)[1] == pytest.approx(10 * 64 * 1000 * 4096 * 36 / 50e9, rel=1e-6)


def test_feasibility_constraints():
    m = model(H_max_bytes=100e9)  # B K_seq = 64 * 4.83 GB = 309 GB -> needs N_D >= 4
    assert [od.feasible_disagg(m, 1, nd) for nd in (1, 3, 4)] == [False, False, True]
    m = model(prefill_tokens_per_worker=200000.0)  # lambda_P = 64 * 10 * 1000 = 640 000 tokens -> N_P >= 4
    assert [od.feasible_disagg(m, n_p, 8) for n_p in (3, 4)] == [False, True]


def enumerate_candidates(m, N):
    cands = {(0, 0, N): od.makespan_coloc(m, N)}
    for n_p in range(1, N):
        if od.feasible_disagg(m, n_p, N - n_p):
            cands[(n_p, N - n_p, 0)] = od.makespan_disagg(m, n_p, N - n_p)[0]
    return cands


def test_decide_is_the_argmin_and_forced_switches_ignore_thresholds():
    m = model(A=0.005, b=2e-3, t_prefill=4e-5, H_max_bytes=100e9)
    N = 12
    cfg, t = od.decide(m, N)
    cands = enumerate_candidates(m, N)
    assert t == min(cands.values()) and cands[cfg] == t
    # a current configuration that no longer fits forces the switch whatever the thresholds
    assert od.decide(m, N, current=(1, 1, 0), ratio_threshold=10.0, mode_threshold=10.0)[0] == cfg
    assert od.decide(m, N, current=(N - 1, 1, 0), ratio_threshold=10.0, mode_threshold=10.0)[0] == cfg  # KV does not fit


# Two hand-evaluated six-worker models for the hysteresis of Sec. 4.3.2 (theta = 0, A = 0, no transfer, no
# environment time, one turn): per turn the prefill work is B dL t_prefill = 6 worker-seconds and the decode work
# r b B = 60 worker-seconds, so Eq. 1 gives 6/6 + 60/6 + T_over = 11 + T_over and Eq. 2-3 give
# max(6 / N_P, 60 / N_D): (1,5) -> 12, (2,4) -> 15, (3,3) -> 20, (4,2) -> 30, (5,1) -> 60.
HAND = dict(B=60.0, S=1.0, r=100.0, dL=100.0, theta=0.0, A=0.0, b=0.01, t_prefill=0.001, T_env=0.0, K_bytes=0.0, BW=1.0,
            K_seq_bytes=0.0, H_max_bytes=1.0)
DISAGG_WINS = dict(HAND, T_over=5.0)   # colocation 16: the argmin is (1, 5, 0) at 12
COLOC_WINS = dict(HAND, T_over=0.0)    # colocation 11: the argmin is colocation


def hysteresis_cases():
    """(model, current, ratio_threshold, mode_threshold, expected configuration, expected makespan)."""
    D, C = model(**DISAGG_WINS), model(**COLOC_WINS)
    return [
        # ratio move inside disaggregation: (2,4) at 15 -> (1,5) at 12, relative gain 3/15 = 0.2;
        # the (large) mode threshold must play no part
        (D, (2, 4, 0), 0.19, 0.9, (1, 5, 0), 12.0),
        (D, (2, 4, 0), 0.21, 0.9, (2, 4, 0), 15.0),
        # colocation -> disaggregation: 16 -> 12, gain 4/16 = 0.25; the ratio threshold must play no part
        (D, (0, 0, 6), 0.9, 0.24, (1, 5, 0), 12.0),
        (D, (0, 0, 6), 0.0, 0.26, (0, 0, 6), 16.0),
        # disaggregation -> colocation: (1,5) at 12 -> 11, gain 1/12 = 0.0833
        (C, (1, 5, 0), 0.9, 0.08, (0, 0, 6), 11.0),
        (C, (1, 5, 0), 0.0, 0.09, (1, 5, 0), 12.0),
        # the best alternative is a refused mode switch (colocation 11 from (3,3) at 20: gain 0.45 < 0.5) while
        # a ratio of the same mode clears its own threshold ((1,5) at 12: gain 0.4 > 0.1): the ratio move is taken
        (C, (3, 3, 0), 0.1, 0.5, (1, 5, 0), 12.0),
        (C, (3, 3, 0), 0.1, 0.44, (0, 0, 6), 11.0),
        (C, (3, 3, 0), 0.41, 0.5, (3, 3, 0), 20.0),
        # among admitted ratios the best one wins, not the nearest: from (4,2) at 30 both (3,3) and (1,5) clear 0.3
        (C, (4, 2, 0), 0.3, 0.9, (1, 5, 0), 12.0),
    ]


def test_hand_models_have_the_intended_minima():
    D, C = model(**DISAGG_WINS), model(**COLOC_WINS)
    want = {(1, 5, 0): 12.0, (2, 4, 0): 15.0, (3, 3, 0): 20.0, (4, 2, 0): 30.0, (5, 1, 0): 60.0}
    for m, coloc in ((D, 16.0), (C, 11.0)):
        cands = enumerate_candidates(m, 6)
        assert cands.pop((0, 0, 6)) == pytest.approx(coloc, rel=1e-14)
        assert set(cands) == set(want)
        for c, t in want.items():
            assert cands[c] == pytest.approx(t, rel=1e-14)
    cfg, t = od.decide(D, 6)
    assert cfg == (1, 5, 0) and cfg[2] == 0 and t == pytest.approx(12.0, rel=1e-14)   # disaggregated argmin
    cfg, t = od.decide(C, 6)
    assert cfg == (0, 0, 6) and t == pytest.approx(11.0, rel=1e-14)                   # colocated argmin


def test_mode_dependent_hysteresis_hand_cases():
    for m, cur, rt, mt, want_cfg, want_t in hysteresis_cases():
        cfg, t = od.decide(m, 6, current=cur, ratio_threshold=rt, mode_threshold=mt)
        assert cfg == want_cfg, (cur, rt, mt, cfg)
        assert t == pytest.approx(want_t, rel=1e-14)


# Two workers, every quantity a power of two, so the comparison at the threshold is exact in binary:
# colocation = 8192/2 * 2^-10 + 64 * (2^-6 * 64 / 2) + 92 = 4 + 32 + 92 = 128, (1,1) = max(8, 64) = 64, gain exactly 1/2.
EXACT = dict(B=64.0, S=1.0, r=64.0, dL=128.0, theta=0.0, A=0.0, b=2.0 ** -6, t_prefill=2.0 ** -10, T_over=92.0, T_env=0.0,
             K_bytes=0.0, BW=1.0, K_seq_bytes=0.0, H_max_bytes=1.0)


def test_hysteresis_is_strict_at_the_threshold():
    m = model(**EXACT)
    assert od.makespan_coloc(m, 2) == 128.0 and od.makespan_disagg(m, 1, 1)[0] == 64.0
    assert od.decide(m, 2, current=(0, 0, 2), mode_threshold=0.5) == ((0, 0, 2), 128.0)      # gain == threshold: stay
    assert od.decide(m, 2, current=(0, 0, 2), mode_threshold=0.4375) == ((1, 1, 0), 64.0)
    # relative, not absolute: an absolute reading of 0.4375 s would also pass, one of 60 s would too (64 > 60),
    # while 60 as a fraction of the current makespan can never be exceeded
    assert od.decide(m, 2, current=(0, 0, 2), mode_threshold=60.0)[0] == (0, 0, 2)


def test_change_counts_match_brute_force_minimum():
    rng = np.random.default_rng(3)
    for _ in range(200):
        n, n_roles = int(rng.integers(1, 7)), int(rng.integers(1, 4))
        cur_active = rng.integers(0, 2, n)
        dst_active = rng.integers(0, 2, n)
        cur_role = rng.integers(0, n_roles, n)
        k = int(dst_active.sum())
        cuts = np.sort(rng.integers(0, k + 1, n_roles - 1))
        counts = np.diff(np.concatenate([[0], cuts, [k]])).astype(int)
        dw, dr = od.change_counts(cur_active, cur_role, dst_active, counts)
        assert dw == int((cur_active != dst_active).sum())
        assert dr == od.brute_force_min_role_changes(cur_active, cur_role, dst_active, counts)


def test_toggle_gate_boundary():
    assert od.toggle_gate(32, 64, 100.0, 80.0, 9.99) and not od.toggle_gate(32, 64, 100.0, 80.0, 10.0)
    assert not od.toggle_gate(0, 64, 100.0, 80.0, 0.0)


# ---------------------------------------------------------------- the library's C functions against the oracle

def random_model(rng):
    return model(B=float(rng.integers(8, 257)), S=float(rng.integers(1, 30)), r=float(rng.integers(1, 600)),
                 dL=float(rng.integers(16, 4000)), theta=float(rng.uniform(0, 3)), A=float(rng.uniform(1e-3, 0.05)),
                 b=float(rng.uniform(1e-5, 5e-3)), t_prefill=float(rng.uniform(1e-6, 1e-4)),
                 T_over=float(rng.uniform(0, 0.1)), T_env=float(rng.uniform(0, 30)),
                 K_bytes=float(rng.integers(1, 40) * 4096), BW=float(rng.uniform(1e9, 1e11)),
                 K_seq_bytes=float(rng.uniform(1e8, 8e9)), H_max_bytes=float(rng.uniform(2e10, 1.5e11)),
                 prefill_tokens_per_worker=float(rng.choice([0.0, 5e4, 5e5])))


def test_c_functions_match_the_oracle():
    import paper_2609_35158_b200 as pd

    rng = np.random.default_rng(11)
    for _ in range(300):
        m = random_model(rng)
        cm = c_model(m)
        N = int(rng.integers(2, 33))
        assert pd.pd_makespan_coloc(cm, N) == pytest.approx(od.makespan_coloc(m, N), rel=1e-13)
        n_p = int(rng.integers(1, N))
        got = pd.pd_makespan_disagg(cm, n_p, N - n_p)
        np.testing.assert_allclose(got, od.makespan_disagg(m, n_p, N - n_p), rtol=1e-13)
        assert pd.pd_feasible_disagg(cm, n_p, N - n_p) == od.feasible_disagg(m, n_p, N - n_p)
        cur = None
        if rng.random() < 0.7:
            cur = (0, 0, N) if rng.random() < 0.3 else (n_p, N - n_p, 0)
            if rng.random() < 0.2:
                cur = (1, 1, 0)
        rt, mt = float(rng.choice([0.0, 0.02, 0.1])), float(rng.choice([0.0, 0.05, 0.3]))
        want_cfg, want_t = od.decide(m, N, cur, rt, mt)
        got_t = pd.pd_decide(cm, N, None if cur is None else pd.pd_target(*cur, 0.0), rt, mt)
        assert (got_t.N_P, got_t.N_D, got_t.N_C) == want_cfg
        assert got_t.makespan == pytest.approx(want_t, rel=1e-13)
    assert math.isnan(pd.pd_makespan_coloc(c_model(model(B=-1.0)), 4))


def test_c_decide_hand_cases():
    import paper_2609_35158_b200 as pd

    for m, cur, rt, mt, want_cfg, want_t in hysteresis_cases():
        got = pd.pd_decide(c_model(m), 6, pd.pd_target(*cur, 0.0), rt, mt)
        assert (got.N_P, got.N_D, got.N_C) == want_cfg, (cur, rt, mt)
        assert got.makespan == pytest.approx(want_t, rel=1e-14)
    cm = c_model(model(**EXACT))
    for mt, want in ((0.5, (0, 0, 2)), (0.4375, (1, 1, 0)), (60.0, (0, 0, 2))):
        got = pd.pd_decide(cm, 2, pd.pd_target(0, 0, 2, 0.0), 0.0, mt)
        assert (got.N_P, got.N_D, got.N_C) == want


def test_c_min_change_plan_is_valid_and_minimal():
    import paper_2609_35158_b200 as pd

    rng = np.random.default_rng(12)
    for _ in range(300):
        n, n_roles = int(rng.integers(1, 12)), int(rng.integers(1, 5))
        cur_active = rng.integers(0, 2, n).astype(np.int32)
        dst_active = rng.integers(0, 2, n).astype(np.int32)
        cur_role = rng.integers(0, n_roles, n).astype(np.int32)
        k = int(dst_active.sum())
        cuts = np.sort(rng.integers(0, k + 1, n_roles - 1))
        counts = np.diff(np.concatenate([[0], cuts, [k]])).astype(np.int32)
        new_role, dw, dr = pd.pd_min_change_plan(cur_active, cur_role, dst_active, counts)
        assert (dw, dr) == od.change_counts(cur_active, cur_role, dst_active, counts)
        # the plan is concrete: every target worker has a role, role counts are met, nobody else is touched
        assert np.all((new_role >= 0) == (dst_active != 0))
        assert np.array_equal(np.bincount(new_role[new_role >= 0], minlength=n_roles), counts)
        survivors = (cur_active != 0) & (dst_active != 0)
        assert int((new_role[survivors] != cur_role[survivors]).sum()) == dr  # exactly the minimum switches
    with pytest.raises(pd.PdError):
        pd.pd_min_change_plan([1, 1], [0, 0], [1, 1], [1])  # role counts do not cover the target set


def test_c_gate_and_fit():
    import paper_2609_35158_b200 as pd

    assert pd.pd_toggle_gate(32, 64, 100.0, 80.0, 9.99) and not pd.pd_toggle_gate(32, 64, 100.0, 80.0, 10.0)
    x = np.array([8, 64, 256, 512], dtype=np.float64)
    A, b = pd.pd_fit_decode_cost(x, 0.004 + 7e-6 * x)
    assert A == pytest.approx(0.004, rel=1e-10) and b == pytest.approx(7e-6, rel=1e-10)
    with pytest.raises(pd.PdError):
        pd.pd_fit_decode_cost([1.0, 1.0], [2.0, 3.0])
