"""CPU oracle for the per-layer MoE decode step with adaptive expert prefetch.

TEST INFRASTRUCTURE, NOT PRODUCT.  Plain, slow, fp64 numpy written from the paper; it shares
no code with the CUDA library and never imports it.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg call it.

Every function follows one passage of the paper, in the paper's notation (Table I):
N experts, k routed per token, delta extra-prefetch budget, K_r routed set, K_p prefetched
set, delta* oracle budget, delta_hat selected budget, tau coverage target, p_delta coverage
probability, w / theta the ordinal-logistic parameters.  Equations are numbered in order of
appearance: (1) K_p^(delta), (2) coverage predicate, (3) delta*, (4)-(5) objective,
(6)-(7) CDF, (8) ordinal logistic model, (9) runtime budget, (10) KL, (11) CDF loss,
(12) prefetch-overlap bound.

Where the paper is silent the reading taken is stated at the function (and listed in the
design notes): all orderings are "value descending, then lower expert index"; decisions are
taken on logits in fp64; the confidence feature x is the prefetch distribution sorted in
descending order; gates are renormalised over the executed set; the HBM cache is a per-layer
slot table with least-recently-stamped replacement.

Parity status: every function here is pinned by tests (closed forms, brute force, library
special cases, invariants) except the *absolute* overlap / mean-budget values the paper
reports for its trained predictors on a public corpus: those are "parity unpinned".
"""
from __future__ import annotations

import math
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

NEAR_TIE_LOGIT = 1e-6       # a deciding logit gap below this is a near-tie
NEAR_TIE_THRESHOLD = 1e-5   # same for the threshold test theta_delta - s >= logit(tau)


# --------------------------------------------------------------------------------------
# Routers (Sec. III-A: router -> softmax over N -> top-k;  Sec. IV-D: the prefetch router
# mirrors the original router: linear layer -> logits -> softmax)
# --------------------------------------------------------------------------------------
def linear_logits(W: np.ndarray, b: Optional[np.ndarray], v: np.ndarray) -> np.ndarray:
    """z[e] = b[e] + sum_i W[e][i] * v[i], accumulated in ascending i, fp64."""
    W = np.asarray(W, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    N, d = W.shape
    z = np.zeros(N, dtype=np.float64) if b is None else np.asarray(b, dtype=np.float64).copy()
    for e in range(N):
        # np.cumsum would fix the order too; math.fsum is exact, which is stricter still.
        z[e] += math.fsum(W[e] * v)
    return z


def softmax(z: np.ndarray) -> np.ndarray:
    """softmax with max subtraction (Sec. IV-D, Alg. 1 line 3)."""
    z = np.asarray(z, dtype=np.float64)
    ez = np.exp(z - z.max())
    return ez / ez.sum()


def rank_desc(z: np.ndarray) -> np.ndarray:
    """Permutation pi: experts sorted by (z descending, index ascending).  pi[j-1] = e_j, the
    ordered list E of Sec. IV-B."""
    z = np.asarray(z, dtype=np.float64)
    return np.array(sorted(range(len(z)), key=lambda e: (-z[e], e)), dtype=np.int64)


def min_adjacent_gap(z: np.ndarray, upto: Optional[int] = None) -> float:
    """Smallest gap between neighbours of z sorted descending, among the first `upto`
    neighbour pairs (all if None): pair j is (position j, position j+1), so upto = m covers the
    order inside the first m positions and the boundary below position m.  Used only to flag
    near-ties."""
    s = np.sort(np.asarray(z, dtype=np.float64))[::-1]
    g = s[:-1] - s[1:]
    if upto is not None:
        g = g[:upto]
    return float(g.min()) if len(g) else float("inf")


def boundary_gap(z: np.ndarray, m: int) -> float:
    """Gap between the m-th and the (m+1)-th largest value of z: the one comparison that decides
    which m elements form the top-m SET.  inf when there is no such boundary (m <= 0 or m >= len)."""
    s = np.sort(np.asarray(z, dtype=np.float64))[::-1]
    if m <= 0 or m >= len(s):
        return float("inf")
    return float(s[m - 1] - s[m])


# --------------------------------------------------------------------------------------
# Prefetch stage (Sec. IV-A stage 1; Sec. IV-C Eq. (8), (9); Eq. (1))
# --------------------------------------------------------------------------------------
def prefetch_scores(W_p, b_p, h):
    """S1: z_p = W_p h + b_p, q_p = softmax(z_p); S2: ranking pi."""
    z_p = linear_logits(W_p, b_p, h)
    return z_p, softmax(z_p), rank_desc(z_p)


def coverage_probabilities(x: np.ndarray, w: np.ndarray, theta: np.ndarray) -> np.ndarray:
    """p_delta(x) = sigma(theta_delta - w^T x), delta = 0..N-k  (Eq. (8))."""
    s = math.fsum(np.asarray(w, np.float64) * np.asarray(x, np.float64))
    t = np.asarray(theta, np.float64) - s
    return 1.0 / (1.0 + np.exp(-t))


def select_budget(q_p: np.ndarray, pi: np.ndarray, w: np.ndarray, theta: np.ndarray,
                  tau: float, k: int, C: int) -> Dict:
    """S3: delta_hat(x) = min{delta : p_delta(x) >= tau}  (Eq. (9)) and K_p = {e_1..e_{k+delta_hat}}
    (Eq. (1)).

    Readings: x = q_p sorted descending (x_j = q_p[pi[j]]); the test p_delta >= tau is taken
    in the logit domain, theta_delta - s >= ln(tau/(1-tau)), which is the same predicate in
    exact arithmetic; tau <= 0 gives delta_hat = 0, tau >= 1 gives N-k; if no delta passes,
    delta_hat = N-k (p_{N-k} is 1 in truth because delta* <= N-k); finally the budget is
    capped to the buffer, delta_hat <- min(delta_hat, C-k).
    """
    N = len(q_p)
    x = np.asarray(q_p, np.float64)[np.asarray(pi)]
    s = math.fsum(np.asarray(w, np.float64) * x)
    theta = np.asarray(theta, np.float64)
    margin = float("inf")
    if tau <= 0.0:
        d_hat = 0
    elif tau >= 1.0:
        d_hat = N - k
    else:
        t_tau = math.log(tau / (1.0 - tau))
        d_hat = N - k
        for delta in range(N - k + 1):
            if theta[delta] - s >= t_tau:
                d_hat = delta
                break
        # only the comparisons that were taken decide delta_hat: delta = 0 .. delta_hat
        margin = float(np.min(np.abs(theta[:d_hat + 1] - s - t_tau)))
    uncapped = d_hat
    d_hat = min(d_hat, C - k)
    return {"delta_hat": d_hat, "uncapped": uncapped, "capped": int(uncapped > d_hat),
            "P": [int(e) for e in pi[:k + d_hat]], "s": s, "threshold_margin": margin}


# --------------------------------------------------------------------------------------
# Execution stage: exact gate (Sec. III-A; Sec. IV-A stage 2)
# --------------------------------------------------------------------------------------
def route_topk(W_r, b_r, h_post, k: int):
    """S4: z_r = W_r h' + b_r; K_r = first k experts by (z_r desc, index asc), in that order;
    alpha = softmax(z_r) over all N experts (Alg. 1 line 3)."""
    z_r = linear_logits(W_r, b_r, h_post)
    order = rank_desc(z_r)
    return z_r, [int(e) for e in order[:k]], softmax(z_r)


# --------------------------------------------------------------------------------------
# Metrics (Eq. (2), (3); overlap accuracy of Sec. III-B, Challenge 1)
# --------------------------------------------------------------------------------------
def oracle_budget(pi: np.ndarray, K_r: Sequence[int], k: int) -> int:
    """delta* = min{delta : K_r subset of K_p^(delta)} = (largest 1-based rank of a routed
    expert in E) - k  (Eq. (3))."""
    pos = {int(e): j + 1 for j, e in enumerate(pi)}
    return max(pos[e] for e in K_r) - k


def overlap_accuracy(K_r: Sequence[int], P: Sequence[int]) -> float:
    """Fraction of routed experts present in the prefetched set."""
    P = set(P)
    return sum(1 for e in K_r if e in P) / len(K_r)


def covered(K_r: Sequence[int], P: Sequence[int]) -> bool:
    """Eq. (2): success iff K_r minus K_p is empty."""
    return set(K_r) <= set(P)


# --------------------------------------------------------------------------------------
# Stall-free execution set (Algorithm 1) and gates
# --------------------------------------------------------------------------------------
def stall_free_set(K_r: Sequence[int], alpha: np.ndarray, K_p: Sequence[int]) -> List[int]:
    """Execution set of the stall-free mode (Sec. IV-E (2), Alg. 1), stated as one ordering: the
    available experts K_p (the paper's prefetched set; with a persistent cache, the resident set)
    are ordered by (routed first, then router weight alpha descending, then index ascending) and
    the first k = |K_r| of them are executed.  Every available routed expert is kept (there are at
    most k of them) and the places of the missing ones go to the best remaining available experts:
    Alg. 1's candidate pool is K_p minus the kept experts and its Top is by (alpha, then index).
    If fewer than k experts are available the set stays short (cannot happen while |K_p| >= k).
    Returned in ascending expert index.  tests/test_oracle_pins.py proves this equal to the
    step-by-step algorithm by brute force over all subsets."""
    alpha = np.asarray(alpha, np.float64)
    routed = set(int(e) for e in K_r)
    order = sorted(set(int(e) for e in K_p), key=lambda e: (0 if e in routed else 1, -alpha[e], e))
    return sorted(order[:len(routed)])


def substitution_margin(z_r: np.ndarray, K_r: Sequence[int], K_p: Sequence[int]) -> float:
    """Near-tie margin of Alg. 1's Top_{|M|}: the logit gap between the last substitute taken
    and the best one left out (the order of alpha is the order of z_r).  inf when nothing is
    substituted or every remaining available expert is taken."""
    routed = set(int(e) for e in K_r)
    avail = set(int(e) for e in K_p)
    n_missing = len(routed - avail)
    pool = sorted(avail - routed)
    if n_missing == 0 or not pool:
        return float("inf")
    return boundary_gap(np.asarray(z_r, np.float64)[pool], n_missing)


def gates(alpha: np.ndarray, K_exec: Sequence[int], norm_topk: bool = True) -> np.ndarray:
    """Weights of the weighted sum.  norm_topk: g_e = alpha_e / sum_{j in K~} alpha_j (so the
    stall-free weights sum to 1); otherwise g_e = alpha_e."""
    a = np.array([float(alpha[e]) for e in K_exec], dtype=np.float64)
    return a / a.sum() if norm_topk else a


# --------------------------------------------------------------------------------------
# Expert FFN and combine (Sec. III-A: experts process the token independently and the outputs
# are combined by a weighted sum).  SwiGLU form, no biases.
# --------------------------------------------------------------------------------------
def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def swiglu_ffn(W_gate, W_up, W_down, v) -> np.ndarray:
    """FFN(v) = W_down ( silu(W_gate v) * (W_up v) );  W_gate, W_up [I][d], W_down [d][I]."""
    v = np.asarray(v, np.float64)
    g = np.asarray(W_gate, np.float64) @ v
    u = np.asarray(W_up, np.float64) @ v
    return np.asarray(W_down, np.float64) @ (silu(g) * u)


def shared_gate_weight(w_sg, h_post) -> float:
    """Weight of a gated shared expert: sigmoid(w_sg . h').  Not part of the paper's configurations (their shared
    experts run with weight 1, Sec. V-A); model families with a per-token sigmoid gate on the shared FFN use this."""
    z = float(np.dot(np.asarray(w_sg, np.float64), np.asarray(h_post, np.float64)))
    return 1.0 / (1.0 + np.exp(-z))


def moe_output(h_post, K_exec: Sequence[int], g: Sequence[float],
               expert_weights: Callable[[int], Tuple[np.ndarray, np.ndarray, np.ndarray]],
               shared=None, shared_gate=None) -> np.ndarray:
    """y = sum_{e in K~, ascending e} g_e FFN_e(h') + s FFN_shared(h'), s = 1 (Sec. V-A) or, with a gate vector
    shared_gate, s = sigmoid(shared_gate . h')."""
    y = np.zeros(len(h_post), dtype=np.float64)
    for e, ge in sorted(zip(K_exec, g)):
        Wg, Wu, Wd = expert_weights(int(e))
        y += float(ge) * swiglu_ffn(Wg, Wu, Wd, h_post)
    if shared is not None:
        s = 1.0 if shared_gate is None else shared_gate_weight(shared_gate, h_post)
        y += s * swiglu_ffn(shared[0], shared[1], shared[2], h_post)
    return y


# --------------------------------------------------------------------------------------
# HBM slot cache (build-defined; the paper's own policy, load-use-evict per layer, is
# cache_reuse=False)
# --------------------------------------------------------------------------------------
class SlotCache:
    """Per-layer table of C slots.  slot_expert[s] is the expert held by slot s (-1 empty),
    expert_slot[e] its inverse (-1 not resident), slot_stamp[s] the step at which the slot was
    last installed or used (-1 never).  A victim is the slot with the smallest
    (stamp, slot index) among slots whose expert is not protected."""

    def __init__(self, N: int, C: int, cache_reuse: bool = True):
        self.N, self.C, self.cache_reuse = N, C, cache_reuse
        self.slot_expert = [-1] * C
        self.expert_slot = [-1] * N
        self.slot_stamp = [-1] * C
        self.clock = 0

    # -- snapshot / restore (lock-step verification, checkpoint) --
    def get_state(self):
        return list(self.expert_slot), list(self.slot_stamp), self.clock

    def set_state(self, expert_slot, slot_stamp, clock):
        self.expert_slot = [int(x) for x in expert_slot]
        self.slot_stamp = [int(x) for x in slot_stamp]
        self.clock = int(clock)
        self.slot_expert = [-1] * self.C
        for e, s in enumerate(self.expert_slot):
            if s >= 0:
                assert self.slot_expert[s] == -1, "two experts in one slot"
                self.slot_expert[s] = e

    def resident(self) -> List[int]:
        return [e for e in range(self.N) if self.expert_slot[e] >= 0]

    def begin_step(self):
        self.clock += 1
        if not self.cache_reuse:
            self.slot_expert = [-1] * self.C
            self.expert_slot = [-1] * self.N
            self.slot_stamp = [-1] * self.C

    def touch(self, e: int):
        self.slot_stamp[self.expert_slot[e]] = self.clock

    def touch_all(self, experts: Sequence[int]):
        """Recency update of a set of resident experts that were executed (stall-free mode: the
        union of the execution sets; order is irrelevant, every stamp becomes the clock)."""
        for e in sorted(set(int(x) for x in experts)):
            self.touch(e)

    def _acquire(self, e: int, protect: set, deprioritise: set) -> Optional[Tuple[int, int]]:
        """Make e resident.  Returns (e, slot) if a copy is needed, None on a hit."""
        if self.expert_slot[e] >= 0:
            self.touch(e)
            return None
        best = None
        for s in range(self.C):
            held = self.slot_expert[s]
            if held >= 0 and held in protect:
                continue
            key = (1 if (held >= 0 and held in deprioritise) else 0, self.slot_stamp[s], s)
            if best is None or key < best[0]:
                best = (key, s)
        if best is None:
            raise RuntimeError("no evictable slot")
        s = best[1]
        if self.slot_expert[s] >= 0:
            self.expert_slot[self.slot_expert[s]] = -1
        self.slot_expert[s] = e
        self.expert_slot[e] = s
        self.slot_stamp[s] = self.clock
        return (e, s)

    def prefetch(self, P_sets: Sequence[Sequence[int]]) -> Tuple[List[int], List[Tuple[int, int]]]:
        """S5.  The prefetch set U is the union of the per-token candidate sets ordered by
        (number of tokens that contain e, descending; expert index ascending), truncated to C.
        Its members are made resident in ascending expert index with U protected, so the slot
        decisions depend on the set U only.  Returns (U sorted ascending, copy list)."""
        count: Dict[int, int] = {}
        for P in P_sets:
            for e in P:
                count[int(e)] = count.get(int(e), 0) + 1
        U = sorted(count, key=lambda e: (-count[e], e))[: self.C]
        U_sorted = sorted(U)
        prot = set(U_sorted)
        copies = []
        for e in U_sorted:
            c = self._acquire(e, prot, set())
            if c is not None:
                copies.append(c)
        return U_sorted, copies

    def demand(self, K_r_sets: Sequence[Sequence[int]]) -> Tuple[List[int], List[List[Tuple[int, int]]]]:
        """Correctness-preserving mode.  Need = union of the routed sets.  Wave 0 is Need that is
        resident (touched).  Missing experts, in ascending index and in chunks of at most C, are
        installed with the chunk protected and members of Need least preferred as victims.
        Returns (missing list, copy list per extra wave)."""
        need = sorted(set(int(e) for K in K_r_sets for e in K))
        need_set = set(need)
        missing = [e for e in need if self.expert_slot[e] < 0]
        for e in need:
            if self.expert_slot[e] >= 0:
                self.touch(e)
        waves = []
        for i in range(0, len(missing), self.C):
            chunk = missing[i:i + self.C]
            prot = set(chunk)
            waves.append([self._acquire(e, prot, need_set) for e in chunk])
        return missing, waves


# --------------------------------------------------------------------------------------
# One layer-step, all tokens of the batch (runtime sequencing of Sec. IV-D: predict + budget before
# attention, prefetch during attention, exact gate after attention, then the chosen execution mode)
# --------------------------------------------------------------------------------------
def layer_step(cache: SlotCache, *, W_p, b_p, W_r, b_r, w, theta, tau: float, k: int,
               h: np.ndarray, h_post: np.ndarray, mode: str,
               expert_weights: Optional[Callable] = None, shared=None, shared_gate=None,
               norm_topk: bool = True, compute_ffn: bool = True, ffn_tokens: Optional[Sequence[int]] = None) -> Dict:
    """h, h_post: [B][d].  mode: 'exact' (correctness-preserving) or 'stall_free'.
    Returns every decision of the step, with the margins needed to flag near-ties.
    ffn_tokens limits the (slow) FFN evaluation to some tokens of the batch; decisions are always
    computed for all."""
    B = h.shape[0]
    N = np.asarray(W_r).shape[0]
    out: Dict = {"B": B, "tokens": []}
    cache.begin_step()
    # prefetch stage
    P_sets = []
    for b in range(B):
        z_p, q_p, pi = prefetch_scores(W_p, b_p, h[b])
        sel = select_budget(q_p, pi, w, theta, tau, k, cache.C)
        # rank_margin decides the whole ranking pi; cand_margin only the ordered candidate list
        # (order inside the first k + delta_hat positions and the boundary below them)
        tok = {"z_p": z_p, "q_p": q_p, "pi": pi, **sel,
               "rank_margin": min_adjacent_gap(z_p),
               "cand_margin": min_adjacent_gap(z_p, upto=k + sel["delta_hat"])}
        out["tokens"].append(tok)
        P_sets.append(sel["P"])
    U, copies = cache.prefetch(P_sets)
    out["U"] = U
    out["prefetch_copies"] = copies
    R = cache.resident()
    out["resident_after_prefetch"] = R
    Rset = set(R)
    # execution stage
    K_sets = []
    for b in range(B):
        tok = out["tokens"][b]
        z_r, K_r, alpha = route_topk(W_r, b_r, h_post[b], k)
        tok.update({"z_r": z_r, "K_r": K_r, "alpha": alpha,
                    "route_margin": min_adjacent_gap(z_r, upto=k),
                    "delta_star": oracle_budget(tok["pi"], K_r, k),
                    "overlap_P": overlap_accuracy(K_r, tok["P"]),
                    "overlap_R": overlap_accuracy(K_r, R),
                    "covered": covered(K_r, tok["P"]),
                    "n_miss": sum(1 for e in K_r if e not in Rset)})
        K_sets.append(K_r)
    if mode == "exact":
        missing, waves = cache.demand(K_sets)
        out["missing"] = missing
        out["demand_copies"] = [c for wv in waves for c in wv]
        for tok in out["tokens"]:
            tok["K_exec"] = sorted(tok["K_r"])
            tok["n_subst"] = 0
            tok["subst_margin"] = float("inf")
    elif mode == "stall_free":
        out["missing"] = []
        out["demand_copies"] = []
        used = set()
        for tok in out["tokens"]:
            tok["K_exec"] = stall_free_set(tok["K_r"], tok["alpha"], R)
            tok["n_subst"] = len(set(tok["K_exec"]) - set(tok["K_r"]))
            tok["subst_margin"] = substitution_margin(tok["z_r"], tok["K_r"], R)
            used |= set(tok["K_exec"])
        cache.touch_all(used)
    else:
        raise ValueError(mode)
    for b, tok in enumerate(out["tokens"]):
        tok["gates"] = gates(tok["alpha"], tok["K_exec"], norm_topk)
        if compute_ffn and expert_weights is not None and (ffn_tokens is None or b in ffn_tokens):
            tok["y"] = moe_output(h_post[b], tok["K_exec"], tok["gates"], expert_weights, shared, shared_gate)
    return out


def near_tie_reasons(tok: Dict) -> List[str]:
    """Which deciding comparisons of one token's step had a margin under the near-tie tolerance:
    'cand' (order or boundary of the candidate list, z_p), 'threshold' (the test of Eq. (9)),
    'route' (order or boundary of K_r, z_r), 'subst' (Alg. 1's Top boundary).  A GPU decision may
    differ from the oracle's only where the matching reason is listed."""
    out = []
    if tok.get("cand_margin", float("inf")) < NEAR_TIE_LOGIT:
        out.append("cand")
    if tok.get("threshold_margin", float("inf")) < NEAR_TIE_THRESHOLD:
        out.append("threshold")
    if tok.get("route_margin", float("inf")) < NEAR_TIE_LOGIT:
        out.append("route")
    if tok.get("subst_margin", float("inf")) < NEAR_TIE_LOGIT:
        out.append("subst")
    return out
