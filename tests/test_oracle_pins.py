"""Pins for the CPU oracle: values the paper prints, closed forms, brute force on tiny inputs,
library special cases and invariants.  None of these re-types an oracle formula: each checks
the oracle against an independent statement of the same fact."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import apex_oracle as ao
from paper_2608_11688_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- values the paper prints
def test_overlap_fraction_examples_from_paper():
    for k, hits, expect in _rows("overlap_fraction.txt"):
        k, hits, expect = int(k), int(hits), float(expect)
        K_r = list(range(k))
        P = list(range(hits)) + [100 + i for i in range(k - hits)]   # same size, one expert wrong
        assert ao.overlap_accuracy(K_r, P) == expect
        assert not ao.covered(K_r, P)


def test_parameter_counts_pin_shapes_of_prefetch_router_and_cdf_model():
    # W_p is d x N and the confidence model has (at most) 2N numbers per layer: x lives in R^N.
    for model, L, d, N, millions in _rows("param_counts.txt"):
        L, d, N = int(L), int(d), int(N)
        cfg = synth.tiny_config(d=d, N=N, k=2, I=8, C=4)
        W_r, b_r, W_p, b_p = synth.router_weights(cfg, 0)
        w, theta = synth.handset_cdf_params(cfg)
        assert W_p.shape == (N, d)
        assert w.shape == (N,) and theta.shape[0] <= N
        total = L * (W_p.size + 2 * N)
        assert f"{total / 1e6:.2f}" == millions, (model, total)


# ---------------------------------------------------------------- library special cases
def test_logits_and_softmax_match_torch_fp64():
    rng = np.random.default_rng(0)
    for N, d in [(8, 64), (40, 1536), (5, 7)]:
        W = rng.standard_normal((N, d)).astype(np.float32)
        b = rng.standard_normal(N).astype(np.float32)
        v = rng.standard_normal(d).astype(np.float32)
        z = ao.linear_logits(W, b, v)
        zt = torch.from_numpy(W).double() @ torch.from_numpy(v).double() + torch.from_numpy(b).double()
        np.testing.assert_allclose(z, zt.numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(ao.softmax(z), torch.softmax(zt, 0).numpy(), rtol=1e-13, atol=0)
    # a transposed operand or a dropped bias would fail the above; no-bias path:
    np.testing.assert_allclose(ao.linear_logits(W, None, v), (torch.from_numpy(W).double() @ torch.from_numpy(v).double()).numpy(), atol=1e-12)


def test_softmax_is_shift_invariant_and_stable():
    z = np.array([1000.0, 999.0, -1000.0])
    q = ao.softmax(z)
    assert np.isfinite(q).all() and abs(q.sum() - 1) < 1e-15
    np.testing.assert_allclose(q, ao.softmax(z - 1000.0), rtol=1e-15)


def test_swiglu_matches_torch_functional_and_zero_gate():
    rng = np.random.default_rng(1)
    d, I = 48, 20
    Wg, Wu = rng.standard_normal((I, d)), rng.standard_normal((I, d))
    Wd = rng.standard_normal((d, I))
    v = rng.standard_normal(d)
    t = lambda a: torch.from_numpy(np.asarray(a))
    ref = t(Wd) @ (torch.nn.functional.silu(t(Wg) @ t(v)) * (t(Wu) @ t(v)))
    np.testing.assert_allclose(ao.swiglu_ffn(Wg, Wu, Wd, v), ref.numpy(), rtol=1e-12, atol=1e-12)
    assert np.all(ao.swiglu_ffn(np.zeros((I, d)), Wu, Wd, v) == 0.0)       # silu(0) = 0
    # N = k = 1: the MoE layer is the plain FFN (the only gate is 1)
    y = ao.moe_output(v, [0], ao.gates(ao.softmax(np.array([0.3])), [0]), lambda e: (Wg, Wu, Wd))
    np.testing.assert_allclose(y, ref.numpy(), rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- ranking and top-k: brute force
def test_rank_desc_against_definition_with_ties():
    rng = np.random.default_rng(2)
    for trial in range(200):
        N = int(rng.integers(1, 9))
        z = rng.integers(-2, 3, size=N).astype(np.float64)      # many duplicates
        pi = ao.rank_desc(z)
        assert sorted(pi) == list(range(N))
        for j, e in enumerate(pi):
            better = sum(1 for f in range(N) if z[f] > z[e] or (z[f] == z[e] and f < e))
            assert better == j


def test_route_topk_bruteforce_subset_and_order():
    rng = np.random.default_rng(3)
    for trial in range(50):
        N, d, k = 7, 16, 3
        W = rng.standard_normal((N, d)); b = rng.standard_normal(N); v = rng.standard_normal(d)
        z, K_r, alpha = ao.route_topk(W, b, v, k)
        # the top-k set maximises the sum of logits over all k-subsets
        best = max(itertools.combinations(range(N), k), key=lambda S: sum(z[list(S)]))
        assert set(best) == set(K_r)
        assert all(z[K_r[i]] >= z[K_r[i + 1]] for i in range(k - 1))
        assert abs(alpha.sum() - 1) < 1e-14 and np.argmax(alpha) == K_r[0]


# ---------------------------------------------------------------- budget selection, Eq. (8)-(9)
def _budget_bruteforce_pdomain(x, w, theta, tau, N, k):
    s = float(np.dot(w.astype(np.float64), x))
    for delta in range(N - k + 1):
        p = 1.0 / (1.0 + math.exp(-(float(theta[delta]) - s)))
        if p >= tau:
            return delta
    return N - k


def test_select_budget_matches_probability_domain_bruteforce():
    rng = np.random.default_rng(4)
    checked = 0
    for trial in range(400):
        N = int(rng.integers(3, 12)); k = int(rng.integers(1, N)); C = N
        q = ao.softmax(rng.standard_normal(N) * 2)
        pi = ao.rank_desc(q)
        w = rng.standard_normal(N).astype(np.float32) * 3
        theta = np.sort(rng.standard_normal(N - k + 1).astype(np.float32) * 2)
        tau = float(rng.uniform(0.05, 0.99))
        sel = ao.select_budget(q, pi, w, theta, tau, k, C)
        if sel["threshold_margin"] < 1e-9:
            continue
        x = np.sort(q)[::-1]
        assert sel["delta_hat"] == _budget_bruteforce_pdomain(x, w, theta, tau, N, k)
        assert sel["P"] == [int(e) for e in pi[:k + sel["delta_hat"]]]
        checked += 1
    assert checked > 300


def test_select_budget_limits_static_and_cap():
    rng = np.random.default_rng(5)
    N, k = 10, 3
    q = ao.softmax(rng.standard_normal(N)); pi = ao.rank_desc(q)
    w = rng.standard_normal(N).astype(np.float32)
    theta = np.sort(rng.standard_normal(N - k + 1)).astype(np.float32)
    assert ao.select_budget(q, pi, w, theta, 0.0, k, N)["delta_hat"] == 0
    assert ao.select_budget(q, pi, w, theta, 1e-300, k, N)["delta_hat"] == 0
    assert ao.select_budget(q, pi, w, theta, 1.0, k, N)["delta_hat"] == N - k
    for C in (k, 5, N):
        sel = ao.select_budget(q, pi, w, theta, 1.0 - 1e-16, k, C)
        assert sel["delta_hat"] == min(N, C) - k and len(sel["P"]) == min(N, C)
        assert sel["capped"] == int(C < N)
    # w = 0: the budget does not depend on the token (static over-fetch baseline)
    w0 = np.zeros(N, np.float32)
    d0 = {ao.select_budget(ao.softmax(rng.standard_normal(N)), pi, w0, theta, 0.7, k, N)["delta_hat"] for _ in range(20)}
    assert len(d0) == 1


def test_candidate_sets_are_nested_in_tau_and_probabilities_monotone():
    rng = np.random.default_rng(6)
    for trial in range(100):
        N, k = 16, 4
        q = ao.softmax(rng.standard_normal(N) * 1.5); pi = ao.rank_desc(q)
        w = rng.standard_normal(N).astype(np.float32) * 2
        theta = np.sort(rng.standard_normal(N - k + 1)).astype(np.float32) * 2
        p = ao.coverage_probabilities(q[pi], w, theta)
        assert np.all(np.diff(p) >= 0)                                   # Eq. (7)
        prev = None
        for tau in (0.3, 0.6, 0.75, 0.9, 0.97):
            P = ao.select_budget(q, pi, w, theta, tau, k, N)["P"]
            if prev is not None:
                assert P[:len(prev)] == prev                              # nested prefixes of E
            prev = P


# ---------------------------------------------------------------- delta*, coverage
def test_oracle_budget_closed_form_vs_definition():
    rng = np.random.default_rng(7)
    for trial in range(300):
        N = int(rng.integers(2, 12)); k = int(rng.integers(1, N + 1))
        pi = rng.permutation(N)
        K_r = [int(e) for e in rng.choice(N, size=k, replace=False)]
        # Eq. (3) literally: smallest delta whose prefix of E contains K_r
        brute = next(dl for dl in range(N - k + 1) if set(K_r) <= set(int(e) for e in pi[:k + dl]))
        assert ao.oracle_budget(pi, K_r, k) == brute
        for d_hat in range(N - k + 1):                                     # full coverage iff d_hat >= delta*
            assert ao.covered(K_r, pi[:k + d_hat]) == (d_hat >= brute)


def test_identical_routers_and_states_need_no_extra_budget():
    cfg = synth.tiny_config(d=64, N=12, k=3, I=8, C=6)
    W_r, b_r, _, _ = synth.router_weights(cfg, 0)
    h, _ = synth.hidden_states(cfg, 0, T=10)
    for t in range(10):
        z_p, q_p, pi = ao.prefetch_scores(W_r, b_r, h[t, 0])
        _, K_r, _ = ao.route_topk(W_r, b_r, h[t, 0], cfg.k)
        assert ao.oracle_budget(pi, K_r, cfg.k) == 0
        assert ao.overlap_accuracy(K_r, pi[:cfg.k]) == 1.0


# ---------------------------------------------------------------- Algorithm 1
def test_stall_free_set_bruteforce_over_all_subsets():
    rng = np.random.default_rng(8)
    for trial in range(300):
        N = int(rng.integers(3, 7)); k = int(rng.integers(1, N))
        alpha = ao.softmax(rng.standard_normal(N))
        K_r = [int(e) for e in ao.rank_desc(alpha)[:k]]
        size_R = int(rng.integers(k, N + 1))
        R = sorted(int(e) for e in rng.choice(N, size=size_R, replace=False))
        K = ao.stall_free_set(K_r, alpha, R)
        assert len(K) == k and set(K) <= set(R) and (set(K_r) & set(R)) <= set(K)
        if set(K_r) <= set(R):
            assert set(K) == set(K_r)
        # independent characterisation: among all k-subsets of R that keep the available routed
        # experts, Algorithm 1 picks the one of largest total router weight
        keep = set(K_r) & set(R)
        best = max((S for S in itertools.combinations(R, k) if keep <= set(S)),
                   key=lambda S: sum(alpha[list(S)]))
        assert set(best) == set(K)
        g = ao.gates(alpha, K)
        assert abs(g.sum() - 1.0) < 1e-14 and np.all(g > 0)


def test_stall_free_tie_break_prefers_lower_index():
    alpha = np.array([0.4, 0.1, 0.1, 0.1, 0.3])
    assert ao.stall_free_set([0, 4], alpha, [0, 1, 2, 3]) == [0, 1]
    assert ao.stall_free_set([0, 4], alpha, [0, 2, 3]) == [0, 2]


def _algorithm1_stepwise(K_r, alpha, avail):
    """Alg. 1 as a procedure over sets, written for this test only: all routed experts available -> K_r; otherwise the
    available routed ones stay and each missing one is replaced by the best expert (alpha, then lower index) still in
    the pool of available, not yet chosen experts -- one replacement at a time."""
    avail = set(avail)
    chosen = [e for e in K_r if e in avail]
    n_missing = len(K_r) - len(chosen)
    for _ in range(n_missing):
        pool = [e for e in avail if e not in chosen]
        if not pool:
            break
        best = pool[0]
        for e in pool[1:]:
            if alpha[e] > alpha[best] or (alpha[e] == alpha[best] and e < best):
                best = e
        chosen.append(best)
    return sorted(chosen)


def test_stall_free_set_equals_algorithm1_taken_step_by_step():
    rng = np.random.default_rng(81)
    for trial in range(500):
        N = int(rng.integers(2, 10)); k = int(rng.integers(1, N + 1))
        # coarse values: many equal weights, so the index tie-break is exercised
        alpha = rng.integers(1, 5, size=N).astype(np.float64); alpha /= alpha.sum()
        K_r = [int(e) for e in ao.rank_desc(alpha)[:k]]
        R = sorted(int(e) for e in rng.choice(N, size=int(rng.integers(1, N + 1)), replace=False))
        assert ao.stall_free_set(K_r, alpha, R) == _algorithm1_stepwise(K_r, alpha, R)


# ---------------------------------------------------------------- near-tie margins (they decide what the parity harness forgives)
def test_min_adjacent_gap_is_the_closest_pair_and_respects_upto():
    rng = np.random.default_rng(82)
    for trial in range(300):
        n = int(rng.integers(2, 10))
        z = rng.standard_normal(n) if trial % 3 else rng.integers(-2, 3, size=n).astype(np.float64)
        # all neighbours: the smallest distance between any two entries
        brute = min(abs(z[i] - z[j]) for i in range(n) for j in range(i + 1, n))
        assert ao.min_adjacent_gap(z) == pytest.approx(brute, abs=0)
        # upto = m: pairs whose larger member is among the m largest entries (order inside the top m and its boundary)
        order = [int(e) for e in ao.rank_desc(z)]
        for m in range(0, n + 2):
            top = order[:m]
            pairs = [abs(z[a] - z[b]) for a in top for b in range(n) if b != a]
            expect = min(pairs) if pairs else float("inf")
            assert ao.min_adjacent_gap(z, upto=m) == pytest.approx(expect, abs=0)
    assert ao.min_adjacent_gap(np.array([3.0, 1.0, 3.0])) == 0.0            # duplicated value
    assert ao.min_adjacent_gap(np.array([3.0, 1.0, 3.0, 0.5]), upto=1) == 0.0
    assert ao.min_adjacent_gap(np.array([5.0, 1.0, 1.0]), upto=1) == 4.0    # the tie lies below the first boundary
    assert ao.min_adjacent_gap(np.array([2.0])) == float("inf")


def test_boundary_gap_is_the_margin_of_the_top_m_set():
    rng = np.random.default_rng(83)
    for trial in range(300):
        n = int(rng.integers(1, 9))
        z = rng.standard_normal(n) if trial % 2 else rng.integers(-2, 3, size=n).astype(np.float64)
        order = [int(e) for e in ao.rank_desc(z)]
        for m in range(-1, n + 2):
            inside, outside = order[:max(m, 0)], order[max(m, 0):]
            expect = min((z[a] - z[b] for a in inside for b in outside), default=float("inf"))
            assert ao.boundary_gap(z, m) == pytest.approx(expect, abs=0)
            # moving every entry by less than half the gap cannot change the top-m set
            if 0 < m < n and expect > 1e-9:
                zz = z + rng.uniform(-0.49, 0.49, size=n) * expect
                assert set(int(e) for e in ao.rank_desc(zz)[:m]) == set(inside)


def test_threshold_margin_is_the_distance_to_a_different_budget():
    rng = np.random.default_rng(84)
    flipped = 0
    for trial in range(400):
        N = int(rng.integers(3, 12)); k = int(rng.integers(1, N)); C = N
        q = ao.softmax(rng.standard_normal(N) * 2); pi = ao.rank_desc(q)
        w = rng.standard_normal(N).astype(np.float32) * 3
        theta = np.sort(rng.standard_normal(N - k + 1).astype(np.float32) * 2)
        tau = float(rng.uniform(0.05, 0.99))
        sel = ao.select_budget(q, pi, w, theta, tau, k, C)
        # written out again with python floats: the comparisons Eq. (9) takes are delta = 0 .. delta_hat
        s = sum(float(w[j]) * float(np.sort(q)[::-1][j]) for j in range(N))
        t_tau = math.log(tau / (1.0 - tau))
        brute = min(abs(float(theta[dl]) - s - t_tau) for dl in range(sel["uncapped"] + 1))
        assert sel["threshold_margin"] == pytest.approx(brute, rel=1e-9, abs=1e-12)
        m = sel["threshold_margin"]
        if m < 1e-9:
            continue
        # a shift of the score by less than the margin leaves the budget alone ...
        for sign in (-1.0, 1.0):
            th2 = theta.astype(np.float64) + sign * 0.98 * m
            assert ao.select_budget(q, pi, w, th2, tau, k, C)["delta_hat"] == sel["delta_hat"]
        # ... and a shift just beyond it, in one of the two directions, changes it (unless the budget is the
        # fall-back N - k that is taken when no comparison passes: failing one more comparison changes nothing)
        d2 = {ao.select_budget(q, pi, w, theta.astype(np.float64) + sign * 1.02 * m, tau, k, C)["delta_hat"] for sign in (-1.0, 1.0)}
        if sel["delta_hat"] < N - k:
            assert d2 != {sel["delta_hat"]}
            flipped += 1
    assert flipped > 200
    # comparisons beyond delta_hat are never taken and must not count: a threshold far above sits exactly on the test
    q = ao.softmax(np.array([3.0, 1.0, 0.0, -1.0])); pi = ao.rank_desc(q)
    t_tau = math.log(0.9 / 0.1)
    sel = ao.select_budget(q, pi, np.zeros(4, np.float32), np.array([t_tau + 1.0, t_tau + 2.0, t_tau + 2.0 + 1e-9]), 0.9, 1, 4)
    assert sel["delta_hat"] == 0 and sel["threshold_margin"] == pytest.approx(1.0)


def test_substitution_margin_and_near_tie_reasons():
    rng = np.random.default_rng(85)
    for trial in range(300):
        N = int(rng.integers(3, 9)); k = int(rng.integers(1, N))
        z = rng.standard_normal(N) if trial % 2 else rng.integers(-2, 3, size=N).astype(np.float64)
        alpha = ao.softmax(z)
        K_r = [int(e) for e in ao.rank_desc(z)[:k]]
        R = sorted(int(e) for e in rng.choice(N, size=int(rng.integers(k, N + 1)), replace=False))
        K = ao.stall_free_set(K_r, alpha, R)
        subs = [e for e in K if e not in K_r]
        left = [e for e in R if e not in K_r and e not in K]
        expect = min((z[a] - z[b] for a in subs for b in left), default=float("inf"))
        assert ao.substitution_margin(z, K_r, R) == pytest.approx(expect, abs=0)
    base = {"cand_margin": 1.0, "threshold_margin": 1.0, "route_margin": 1.0, "subst_margin": float("inf"), "rank_margin": 0.0}
    assert ao.near_tie_reasons(base) == []                       # a tie elsewhere in the ranking excuses nothing
    assert ao.near_tie_reasons({**base, "cand_margin": 9e-7}) == ["cand"]
    assert ao.near_tie_reasons({**base, "threshold_margin": 9e-6}) == ["threshold"]
    assert ao.near_tie_reasons({**base, "threshold_margin": 2e-5, "route_margin": 0.0, "subst_margin": 5e-7}) == ["route", "subst"]


def test_layer_step_margins_follow_the_deciding_positions():
    # a tie far down the prefetch ranking and one far down the router's ranking: neither decides anything
    N, k, d = 8, 2, 8
    W = np.zeros((N, d), np.float32)
    for e, v in enumerate([5.0, 4.0, 3.0, 2.0, 1.0, 0.5, 0.0, 0.0]):       # experts 6 and 7 tie at the bottom
        W[e, 0] = v
    h = np.zeros((1, d), np.float32); h[0, 0] = 1.0
    cache = ao.SlotCache(N, 4)
    out = ao.layer_step(cache, W_p=W, b_p=None, W_r=W, b_r=None, w=np.zeros(N, np.float32),
                        theta=np.linspace(-1, 5, N - k + 1).astype(np.float32), tau=0.6, k=k, h=h, h_post=h, mode="stall_free",
                        compute_ffn=False)
    tok = out["tokens"][0]
    assert tok["rank_margin"] == 0.0 and tok["cand_margin"] == 1.0 and tok["route_margin"] == 1.0
    assert ao.near_tie_reasons(tok) == []


# ---------------------------------------------------------------- slot cache
def test_slot_cache_hand_traced_example():
    # N=4, C=2.  Traced by hand from the replacement rule (smallest (stamp, slot) not protected).
    c = ao.SlotCache(4, 2)
    c.begin_step()                              # clock 1
    U, cp = c.prefetch([[2, 0]])                # both slots empty: ascending expert order 0->slot0, 2->slot1
    assert U == [0, 2] and cp == [(0, 0), (2, 1)] and c.expert_slot == [0, -1, 1, -1]
    miss, waves = c.demand([[0, 3]])            # 3 missing; victim must not be a Need member if possible: slot1 (expert 2)
    assert miss == [3] and waves == [[(3, 1)]] and c.expert_slot == [0, -1, -1, 1]
    c.begin_step()                              # clock 2
    U, cp = c.prefetch([[3, 1]])                # 3 hit (touched, stamp 2); 1 -> victim slot0 (stamp 1)
    assert cp == [(1, 0)] and c.expert_slot == [-1, 0, -1, 1] and c.slot_stamp == [2, 2]
    miss, waves = c.demand([[1, 3]])
    assert miss == [] and waves == []
    c.begin_step()                              # clock 3
    U, cp = c.prefetch([[1]])                   # hit only: slot0 stamp 3
    assert cp == [] and c.slot_stamp == [3, 2]
    miss, waves = c.demand([[0, 2]])            # both missing, C=2: one chunk; 0 -> slot1 (stamp 2 < 3), 2 -> slot0
    assert miss == [0, 2] and waves == [[(0, 1), (2, 0)]] and c.expert_slot == [1, -1, 0, -1]
    # stall-free steps issue no demand copy; the executed experts are stamped instead.  Traced by hand:
    c = ao.SlotCache(4, 3)
    c.begin_step()                              # clock 1
    c.prefetch([[0, 1, 2]])                     # slots 0, 1, 2 <- experts 0, 1, 2, all stamped 1
    c.begin_step()                              # clock 2
    U, cp = c.prefetch([[1]])                   # hit: slot1 stamp 2
    c.touch_all([2, 1])                         # executed set {1, 2} (a substitute included): slots 1, 2 stamped 2
    assert cp == [] and c.slot_stamp == [1, 2, 2]
    c.begin_step()                              # clock 3
    U, cp = c.prefetch([[3]])                   # the one slot not used last step (slot0, expert 0) is the victim
    assert cp == [(3, 0)] and c.expert_slot == [-1, 1, 2, 0] and c.slot_stamp == [3, 2, 2]


def test_stall_free_step_stamps_exactly_the_executed_experts():
    cfg = synth.tiny_config(d=64, N=10, k=3, I=16, C=6, T=30, sigma_p=1.5)
    W_r, b_r, W_p, b_p = synth.router_weights(cfg, 0)
    w, theta = synth.handset_cdf_params(cfg)
    h, hp = synth.hidden_states(cfg, 0, cfg.T, B=2)
    cache = ao.SlotCache(cfg.N, cfg.C)
    for t in range(cfg.T):
        out = ao.layer_step(cache, W_p=W_p, b_p=b_p, W_r=W_r, b_r=b_r, w=w, theta=theta, tau=0.5, k=cfg.k, h=h[t],
                            h_post=hp[t], mode="stall_free", compute_ffn=False)
        used = set(e for tok in out["tokens"] for e in tok["K_exec"])
        planned = set(out["U"])
        for e in cache.resident():
            stamp = cache.slot_stamp[cache.expert_slot[e]]
            assert (stamp == cache.clock) == (e in used or e in planned), (t, e)


def test_slot_cache_invariants_random_walk():
    rng = np.random.default_rng(9)
    for reuse in (True, False):
        N, C, k = 12, 5, 3
        c = ao.SlotCache(N, C, cache_reuse=reuse)
        for step in range(200):
            c.begin_step()
            P = [int(e) for e in rng.choice(N, size=int(rng.integers(k, C + 1)), replace=False)]
            U, copies = c.prefetch([P])
            assert set(P) <= set(c.resident())                       # nothing needed was evicted
            if not reuse:
                assert len(copies) == len(P)                          # load-use-evict: every candidate is copied
            K_r = [int(e) for e in rng.choice(N, size=k, replace=False)]
            missing, waves = c.demand([K_r])
            assert set(K_r) <= set(c.resident())
            assert sorted(e for wv in waves for e, _ in wv) == sorted(missing)
            for e, s in enumerate(c.expert_slot):                     # tables are mutually inverse
                if s >= 0:
                    assert c.slot_expert[s] == e
            for s, e in enumerate(c.slot_expert):
                if e >= 0:
                    assert c.expert_slot[e] == s
            assert sum(1 for e in c.slot_expert if e >= 0) <= C


def test_full_size_cache_copies_each_expert_once():
    rng = np.random.default_rng(10)
    N = C = 8
    c = ao.SlotCache(N, C)
    seen, total = set(), 0
    for step in range(100):
        c.begin_step()
        P = [int(e) for e in rng.choice(N, size=4, replace=False)]
        _, cp = c.prefetch([P])
        K_r = [int(e) for e in rng.choice(N, size=2, replace=False)]
        _, waves = c.demand([K_r])
        for e, _ in cp + [x for wv in waves for x in wv]:
            assert e not in seen
            seen.add(e); total += 1
    assert total == len(seen) <= N


def test_batched_prefetch_union_order_and_truncation():
    c = ao.SlotCache(10, 3)
    c.begin_step()
    # counts: 5 -> 3 tokens, 1 -> 2, 7 -> 2, 0 -> 1, 9 -> 1 ; keep the 3 most wanted, ties by lower index
    U, cp = c.prefetch([[5, 1, 0], [5, 7, 1], [5, 7, 9]])
    assert U == [1, 5, 7] and [e for e, _ in cp] == [1, 5, 7]


# ---------------------------------------------------------------- whole layer-step
def _dense_topk_moe(W_r, b_r, hp, k, experts, shared, renormalise=True):
    """Written separately from the oracle, with torch fp64 ops: standard MoE layer that knows
    nothing about prefetching or caches (softmax over all experts, top-k; gates renormalised over
    the selected experts, or -- the other convention in use -- the plain softmax values)."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    logits = t(W_r) @ t(hp) + t(b_r)
    probs = torch.softmax(logits, 0)
    top = torch.topk(logits, k).indices
    gate = probs[top] / probs[top].sum() if renormalise else probs[top]
    y = torch.zeros(len(hp), dtype=torch.float64)
    for g, e in zip(gate, top):
        Wg, Wu, Wd = (t(m) for m in experts(int(e)))
        y += g * (Wd @ (torch.nn.functional.silu(Wg @ t(hp)) * (Wu @ t(hp))))
    if shared is not None:
        Wg, Wu, Wd = (t(m) for m in shared)
        y += Wd @ (torch.nn.functional.silu(Wg @ t(hp)) * (Wu @ t(hp)))
    return y.numpy()


def _tiny_problem(cfg, layer=0):
    W_r, b_r, W_p, b_p = synth.router_weights(cfg, layer)
    store = synth.bf16_to_f32_numpy(synth.expert_store(cfg, layer))
    experts = lambda e: synth.split_store(store[e])
    sh = synth.shared_expert(cfg, layer)
    shared = None
    if sh is not None:
        s = synth.bf16_to_f32_numpy(sh)
        shared = synth.split_store(s)
    w, theta = synth.handset_cdf_params(cfg)
    return W_r, b_r, W_p, b_p, experts, shared, w, theta


@pytest.mark.parametrize("reuse", [True, False])
@pytest.mark.parametrize("tau,C", [(0.0, 2), (0.6, 3), (0.9, 5), (1.0, 8)])
def test_exact_mode_equals_dense_topk_moe(tau, C, reuse):
    cfg = synth.tiny_config(d=64, N=8, k=2, I=16, C=C, T=6, I_shared=8 if C == 5 else 0, zipf_s=1.1)
    W_r, b_r, W_p, b_p, experts, shared, w, theta = _tiny_problem(cfg)
    h, hp = synth.hidden_states(cfg, 0, cfg.T, B=2)
    cache = ao.SlotCache(cfg.N, cfg.C, cache_reuse=reuse)
    for t in range(cfg.T):
        out = ao.layer_step(cache, W_p=W_p, b_p=b_p, W_r=W_r, b_r=b_r, w=w, theta=theta, tau=tau,
                            k=cfg.k, h=h[t], h_post=hp[t], mode="exact", expert_weights=experts, shared=shared)
        for b in range(2):
            ref = _dense_topk_moe(W_r, b_r, hp[t, b], cfg.k, experts, shared)
            np.testing.assert_allclose(out["tokens"][b]["y"], ref, rtol=1e-10, atol=1e-13)
            assert set(out["tokens"][b]["K_exec"]) == set(out["tokens"][b]["K_r"])
        need = set(e for tok in out["tokens"] for e in tok["K_r"])
        if len(need) <= cfg.C:                  # otherwise the waves reuse slots within the step
            assert need <= set(cache.resident())


def test_unnormalised_gates_equal_dense_moe_that_keeps_the_softmax_values():
    cfg = synth.tiny_config(d=64, N=8, k=3, I=16, C=8, T=5, I_shared=8)
    W_r, b_r, W_p, b_p, experts, shared, w, theta = _tiny_problem(cfg)
    h, hp = synth.hidden_states(cfg, 0, cfg.T)
    cache = ao.SlotCache(cfg.N, cfg.C)
    for t in range(cfg.T):
        out = ao.layer_step(cache, W_p=W_p, b_p=b_p, W_r=W_r, b_r=b_r, w=w, theta=theta, tau=0.9, k=cfg.k, h=h[t],
                            h_post=hp[t], mode="exact", expert_weights=experts, shared=shared, norm_topk=False)
        tok = out["tokens"][0]
        ref = _dense_topk_moe(W_r, b_r, hp[t, 0], cfg.k, experts, shared, renormalise=False)
        np.testing.assert_allclose(tok["y"], ref, rtol=1e-10, atol=1e-13)
        assert sum(tok["gates"]) < 1.0 - 1e-6                   # k < N: the weights do not sum to one
        assert not np.allclose(tok["y"], _dense_topk_moe(W_r, b_r, hp[t, 0], cfg.k, experts, shared), rtol=1e-6, atol=1e-9)


def test_gated_shared_expert_against_a_dense_layer_and_its_limits():
    # y(gated) - y(no shared) = sigmoid(w_sg . h') * (y(ungated) - y(no shared)), the sigmoid from torch; a zero gate
    # vector halves the shared FFN; a gate vector far along h' switches it fully on, far against it fully off
    cfg = synth.tiny_config(d=64, N=8, k=3, I=16, C=8, T=4, I_shared=8)
    W_r, b_r, W_p, b_p, experts, shared, w, theta = _tiny_problem(cfg)
    h, hp = synth.hidden_states(cfg, 0, cfg.T)
    rng = np.random.default_rng(5)
    w_sg = rng.standard_normal(cfg.d) / np.sqrt(cfg.d)
    for t in range(cfg.T):
        def run(sh, sg):
            cache = ao.SlotCache(cfg.N, cfg.C)
            out = ao.layer_step(cache, W_p=W_p, b_p=b_p, W_r=W_r, b_r=b_r, w=w, theta=theta, tau=0.9, k=cfg.k, h=h[t],
                                h_post=hp[t], mode="exact", expert_weights=experts, shared=sh, shared_gate=sg)
            return out["tokens"][0]["y"]
        v = hp[t, 0].astype(np.float64)
        y_none, y_plain, y_gated = run(None, None), run(shared, None), run(shared, w_sg)
        s = float(torch.sigmoid(torch.from_numpy(w_sg) @ torch.from_numpy(v)))
        assert 0.05 < s < 0.95
        np.testing.assert_allclose(y_gated - y_none, s * (y_plain - y_none), rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(y_plain, _dense_topk_moe(W_r, b_r, v, cfg.k, experts, shared), rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(run(shared, np.zeros(cfg.d)) - y_none, 0.5 * (y_plain - y_none), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(run(shared, 100.0 * v / (v @ v)), y_plain, rtol=1e-12, atol=1e-14)    # sigmoid(100) = 1
        np.testing.assert_allclose(run(shared, -100.0 * v / (v @ v)), y_none, rtol=0, atol=1e-12 * np.abs(y_plain).max())
    assert ao.shared_gate_weight(np.zeros(4), np.ones(4)) == 0.5


def test_stall_free_equals_exact_when_covered_and_differs_only_by_substitution():
    cfg = synth.tiny_config(d=64, N=10, k=3, I=16, C=5, T=40, sigma_p=1.5)
    W_r, b_r, W_p, b_p, experts, shared, w, theta = _tiny_problem(cfg)
    h, hp = synth.hidden_states(cfg, 0, cfg.T)
    cache = ao.SlotCache(cfg.N, cfg.C)
    n_sub = n_same = 0
    for t in range(cfg.T):
        out = ao.layer_step(cache, W_p=W_p, b_p=b_p, W_r=W_r, b_r=b_r, w=w, theta=theta, tau=0.6,
                            k=cfg.k, h=h[t], h_post=hp[t], mode="stall_free", expert_weights=experts)
        tok = out["tokens"][0]
        R = set(out["resident_after_prefetch"])
        assert out["demand_copies"] == [] and set(tok["K_exec"]) <= R and len(tok["K_exec"]) == cfg.k
        assert abs(sum(tok["gates"]) - 1.0) < 1e-14
        if set(tok["K_r"]) <= R:
            ref = _dense_topk_moe(W_r, b_r, hp[t, 0], cfg.k, experts, None)
            np.testing.assert_allclose(tok["y"], ref, rtol=1e-10, atol=1e-13)
            n_same += 1
        else:
            assert tok["n_subst"] == len(set(tok["K_r"]) - R) > 0
            n_sub += 1
    assert n_sub > 0 and n_same > 0          # the noisy predictor exercises both branches


def test_per_layer_staging_policy_copies_every_candidate():
    # cache_reuse=False is the paper's load-use-evict policy: R = P after the prefetch
    cfg = synth.tiny_config(d=64, N=10, k=3, I=16, C=6, T=10)
    W_r, b_r, W_p, b_p, experts, shared, w, theta = _tiny_problem(cfg)
    h, hp = synth.hidden_states(cfg, 0, cfg.T)
    cache = ao.SlotCache(cfg.N, cfg.C, cache_reuse=False)
    for t in range(cfg.T):
        out = ao.layer_step(cache, W_p=W_p, b_p=b_p, W_r=W_r, b_r=b_r, w=w, theta=theta, tau=0.9,
                            k=cfg.k, h=h[t], h_post=hp[t], mode="stall_free", compute_ffn=False)
        tok = out["tokens"][0]
        assert sorted(out["resident_after_prefetch"]) == sorted(tok["P"])
        assert len(out["prefetch_copies"]) == cfg.k + tok["delta_hat"]


def test_generator_rounds_hidden_states_to_bf16_values():
    cfg = synth.tiny_config()
    h, hp = synth.hidden_states(cfg, 0, 4)
    for a in (h, hp):
        t = torch.from_numpy(a)
        assert torch.equal(t, t.to(torch.bfloat16).to(torch.float32))
    x = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8], dtype=np.float32)    # exact ties: round to even
    np.testing.assert_array_equal(synth.round_to_bf16_values(x), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


# ------------------------------------------------------------------ the CPU fit of the confidence model (Eq. (8), (11))
def _cumulative_bce(X, dstar, w, theta):
    """Eq. (11) written out with plain loops: mean over tokens of the sum over thresholds of the binary
    cross-entropy between [delta >= delta*] and sigmoid(theta_delta - w.x)."""
    total = 0.0
    for t in range(X.shape[0]):
        s = float(np.dot(w, X[t]))
        for dl in range(len(theta)):
            z = theta[dl] - s
            y = 1.0 if dl >= dstar[t] else 0.0
            # -[y log p + (1 - y) log(1 - p)] with p = sigmoid(z), in the form that survives p = 1 in fp64
            total += float(np.logaddexp(0.0, z)) - y * z
    return total / X.shape[0]


def _planted_ordinal_data(T, N, k, seed):
    """Tokens whose delta* is drawn from a known ordinal-logistic model: P(delta* <= delta | x) = sigmoid(theta*_delta - w*.x)."""
    rng = np.random.default_rng(seed)
    X = np.sort(rng.dirichlet(np.full(N, 0.6), size=T), axis=1)[:, ::-1].copy()
    w_true = np.zeros(N)
    w_true[:k] = -3.0
    w_true[k:2 * k] = 5.0
    nth = N - k + 1
    theta_true = -1.5 + 0.7 * np.arange(nth)
    theta_true[-1] = 40.0                                   # delta* <= N-k always
    cdf = 1.0 / (1.0 + np.exp(-(theta_true[None, :] - (X @ w_true)[:, None])))
    u = rng.random(T)
    dstar = (u[:, None] > cdf).sum(1)                        # smallest delta with cdf >= u
    return X, dstar.astype(np.int64), w_true, theta_true


def test_cdf_fit_lowers_the_loss_of_eq11_and_recovers_a_planted_model():
    from oracle import fit_cdf
    N, k = 10, 2
    X, dstar, w_true, theta_true = _planted_ordinal_data(6000, N, k, seed=5)
    w0 = np.zeros(N)
    cdf0 = np.clip((np.arange(N - k + 1)[None, :] >= dstar[:, None]).mean(0), 1e-3, 1 - 1e-3)
    th0 = np.log(cdf0 / (1 - cdf0))
    w, theta = fit_cdf.fit(X, dstar, N, k, iters=600)
    assert np.all(np.diff(theta) >= 0)
    sub = slice(0, 1500)                                     # the plain-loop loss on a subset (seconds)
    l_init = _cumulative_bce(X[sub], dstar[sub], w0, th0)
    l_fit = _cumulative_bce(X[sub], dstar[sub], w.astype(np.float64), theta.astype(np.float64))
    l_true = _cumulative_bce(X[sub], dstar[sub], w_true, theta_true)
    assert l_fit < l_init - 0.03 * abs(l_init), (l_init, l_fit, l_true)   # the x-dependence is learnt: better than the marginal CDF
    assert l_fit < l_true + 0.02 * abs(l_true), (l_init, l_fit, l_true)   # and about as good as the model that generated the data
    # the fitted conditional CDF is close to the planted one on fresh tokens
    Xt, _, _, _ = _planted_ordinal_data(2000, N, k, seed=6)
    p_fit = 1.0 / (1.0 + np.exp(-(theta[None, :-1].astype(np.float64) - (Xt @ w.astype(np.float64))[:, None])))
    p_true = 1.0 / (1.0 + np.exp(-(theta_true[None, :-1] - (Xt @ w_true)[:, None])))
    assert np.abs(p_fit - p_true).mean() < 0.03
    # a dropped or sign-flipped gradient term would leave w at zero or drive it the wrong way
    assert np.corrcoef(w[:2 * k], w_true[:2 * k])[0, 1] > 0.9


def test_cdf_fit_without_signal_returns_the_empirical_distribution():
    # x carries no information (all tokens share one x): the optimum of Eq. (11) is the empirical CDF of delta*,
    # theta_delta - w.x = logit(fraction of tokens with delta* <= delta)
    from oracle import fit_cdf
    N, k, T = 8, 3, 3000
    rng = np.random.default_rng(9)
    X = np.tile(np.sort(rng.dirichlet(np.ones(N)))[::-1], (T, 1))
    dstar = rng.integers(0, N - k + 1, size=T)
    w, theta = fit_cdf.fit(X, dstar, N, k, iters=600)
    frac = (np.arange(N - k + 1)[None, :] >= dstar[:, None]).mean(0)
    z = theta.astype(np.float64) - float(X[0] @ w.astype(np.float64))
    np.testing.assert_allclose(1.0 / (1.0 + np.exp(-z[:-1])), frac[:-1], atol=2e-3)


# ------------------------------------------------------------------ the CPU distillation of the prefetch router (Eq. (10))
def _distill_problem(T, N, d, seed, noise=0.0):
    rng = np.random.default_rng(seed)
    W_true = rng.standard_normal((N, d)) / np.sqrt(d)
    b_true = 0.3 * rng.standard_normal(N)
    H = rng.standard_normal((T, d))
    Hp = H + noise * rng.standard_normal((T, d))
    Z = Hp @ W_true.T + b_true
    Z -= Z.max(1, keepdims=True)
    Qr = np.exp(Z)
    Qr /= Qr.sum(1, keepdims=True)
    return H, Qr, W_true, b_true


def test_kl_loss_is_the_definition_and_vanishes_at_the_teacher():
    from oracle import distill
    H, Qr, W_true, b_true = _distill_problem(40, 5, 7, seed=1)
    assert abs(distill.kl_loss(H, Qr, W_true, b_true)) < 1e-12
    rng = np.random.default_rng(2)
    W, b = rng.standard_normal((5, 7)), rng.standard_normal(5)
    total = 0.0
    for t in range(40):                                   # Eq. (10), term by term
        z = W @ H[t] + b
        qp = np.exp(z - z.max())
        qp /= qp.sum()
        total += sum(Qr[t, i] * math.log(Qr[t, i] / qp[i]) for i in range(5))
    assert abs(distill.kl_loss(H, Qr, W, b) - total / 40) < 1e-12 and total > 0


def test_distillation_first_step_follows_the_numerical_gradient():
    # Adam's first step is -lr * sign(gradient): compare it with central differences of the loss.  A transposed
    # operand, a wrong sign or a dropped bias term in the gradient would flip signs here.
    from oracle import distill
    H, Qr, _, _ = _distill_problem(60, 4, 6, seed=3, noise=0.3)
    rng = np.random.default_rng(4)
    W0, b0 = 0.5 * rng.standard_normal((4, 6)), 0.5 * rng.standard_normal(4)
    lr = 1e-3
    W1, b1 = distill.distill(H, Qr, W0, b0, iters=1, lr=lr)
    eps = 1e-6
    for (arr0, arr1) in ((W0, W1), (b0, b1)):
        for idx in np.ndindex(arr0.shape):
            def loss_at(delta):
                Wc, bc = W0.copy(), b0.copy()
                (Wc if arr0 is W0 else bc)[idx] += delta
                return distill.kl_loss(H, Qr, Wc, bc)
            g = (loss_at(eps) - loss_at(-eps)) / (2 * eps)
            if abs(g) > 1e-6:
                np.testing.assert_allclose(arr1[idx] - arr0[idx], -lr * np.sign(g), rtol=1e-3)


def test_distillation_recovers_the_teacher_when_both_see_the_same_state():
    from oracle import distill
    H, Qr, W_true, b_true = _distill_problem(1500, 8, 24, seed=5)
    W0, b0 = np.zeros((8, 24)), np.zeros(8)
    l0 = distill.kl_loss(H, Qr, W0, b0)
    W, b = distill.distill(H, Qr, W0, b0, iters=400, lr=0.02)
    l1 = distill.kl_loss(H, Qr, W, b)
    assert l1 < 0.02 * l0
    Zs, Zt = H @ W.T + b, H @ W_true.T + b_true
    assert (Zs.argmax(1) == Zt.argmax(1)).mean() > 0.97
