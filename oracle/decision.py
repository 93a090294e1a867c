"""Oracle for the PD decision engine: the paper's formulas written out in plain Python.

TEST INFRASTRUCTURE ONLY (same rules as the rest of ``oracle/``). Eq. 1 (colocated makespan), Eq. 2-3
(disaggregated decode / prefill paths, T_dis = max + T_env), the capacity constraints of Sec. 4.2, the
enumeration with mode-dependent hysteresis of Sec. 4.3.2, the change counts of Eq. 5-6 (with a brute-force
minimum over every role assignment for tiny inputs) and the toggle gate of Eq. 7. Models are plain dicts
with the paper's symbol names.
"""
from __future__ import annotations

import itertools


def makespan_coloc(m: dict, N: int) -> float:
    """Eq. 1."""
    per_turn = (m["B"] * m["dL"] / N) * m["t_prefill"] + m["r"] * (m["A"] + m["b"] * m["B"] / N) + m["T_over"]
    return m["S"] * per_turn + m["T_env"]


def makespan_disagg(m: dict, N_P: int, N_D: int):
    """Eq. 2, Eq. 3 and T_dis = max(T_prefill, T_decode) + T_env. Returns (T_dis, T_prefill, T_decode)."""
    f = 1.0 + m["theta"]
    t_decode = m["S"] * m["r"] * (m["A"] + m["b"] * m["B"] / (N_D * f)) * f
    t_prefill = m["S"] * ((m["B"] * m["dL"] / N_P) * m["t_prefill"] + m["B"] * m["dL"] * m["K_bytes"] / m["BW"])
    return max(t_prefill, t_decode) + m["T_env"], t_prefill, t_decode


def feasible_disagg(m: dict, N_P: int, N_D: int) -> bool:
    """Sec. 4.2: the decode pool holds the batch's KV cache; the prefill pool absorbs B S dL tokens per step."""
    if m["B"] * m["K_seq_bytes"] > N_D * m["H_max_bytes"]:
        return False
    cap = m.get("prefill_tokens_per_worker", 0.0)
    if cap > 0 and m["B"] * m["S"] * m["dL"] > N_P * cap:
        return False
    return True


def decide(m: dict, N_k: int, current=None, ratio_threshold=0.0, mode_threshold=0.0):
    """Sec. 4.3.2. Configurations are (N_P, N_D, N_C) tuples; returns (configuration, predicted makespan).

    Without a current configuration: the argmin over colocation and every feasible split. With one that is
    still realisable, hysteresis: an alternative is admitted only if its predicted makespan is lower than the
    current one by more than a threshold, taken here as a fraction of the current makespan, strictly;
    alternatives in the other mode (colocation <-> disaggregation) answer to ``mode_threshold``, other ratios
    of the same mode to ``ratio_threshold``. Every alternative is judged by its own threshold and the best
    admitted one wins, so a refused mode switch does not block a ratio adjustment that clears the smaller
    threshold. A current configuration that cannot be kept forces the switch to the argmin."""
    cands = [((0, 0, N_k), makespan_coloc(m, N_k))]
    for n_p in range(1, N_k):
        if feasible_disagg(m, n_p, N_k - n_p):
            cands.append(((n_p, N_k - n_p, 0), makespan_disagg(m, n_p, N_k - n_p)[0]))
    best, t_best = cands[0]
    for c, t in cands[1:]:  # first strict improvement wins ties, colocation first, then ascending N_P
        if t < t_best:
            best, t_best = c, t
    if current is None:
        return best, t_best
    cur_coloc = current[2] > 0
    cur_ok = sum(current) == N_k and ((current[0] == 0 and current[1] == 0) if cur_coloc
                                      else feasible_disagg(m, current[0], current[1]))
    if not cur_ok:
        return best, t_best  # forced switch: the current topology cannot be kept
    t_cur = makespan_coloc(m, N_k) if cur_coloc else makespan_disagg(m, current[0], current[1])[0]
    choice, t_choice = tuple(current), t_cur
    for c, t in cands:  # same order as above, so ties between admitted alternatives resolve the same way
        if c == tuple(current):
            continue
        threshold = mode_threshold if (c[2] > 0) != cur_coloc else ratio_threshold
        admitted = t_cur - t > threshold * t_cur
        if admitted and t < t_choice:
            choice, t_choice = c, t
    return choice, t_choice


def change_counts(cur_active, cur_role, dst_active, dst_role_count):
    """Eq. 5 and Eq. 6."""
    n = len(cur_active)
    d_worker = sum(1 for w in range(n) if bool(cur_active[w]) != bool(dst_active[w]))
    d_role = 0
    for r, n_dst in enumerate(dst_role_count):
        n_src = sum(1 for w in range(n) if cur_active[w] and dst_active[w] and cur_role[w] == r)
        d_role += n_src - min(n_src, n_dst)
    return d_worker, d_role


def brute_force_min_role_changes(cur_active, cur_role, dst_active, dst_role_count):
    """Minimum number of surviving workers that change role over EVERY assignment of roles to the target
    set that meets the role counts (tiny inputs only)."""
    n = len(cur_active)
    targets = [w for w in range(n) if dst_active[w]]
    roles = [r for r, c in enumerate(dst_role_count) for _ in range(c)]
    assert len(roles) == len(targets)
    best = None
    for perm in set(itertools.permutations(roles)):
        switches = sum(1 for w, r in zip(targets, perm) if cur_active[w] and cur_role[w] != r)
        best = switches if best is None else min(best, switches)
    return best


def toggle_gate(R, B, T_ded, T_full, T_toggle) -> bool:
    """Eq. 7."""
    return (R / B) * (T_ded - T_full) > T_toggle
