"""Offline fit of the ordinal-logistic confidence model (Eq. (8)) by the cumulative binary
cross-entropy of Eq. (11), on synthetic calibration tokens.

TEST / DATA-PREPARATION INFRASTRUCTURE: calls only the CPU oracle and the seeded generators.  Writes
``paper_2608_11688_b200/data/cdf_cfg<id>.npz`` (w [L][N], theta [L][N-k+1], fp32), the frozen
parameters every later run loads -- the analogue of the paper's "CDF model fitted on a held-out
validation set" (Sec. V-A), with the synthetic generator standing in for the corpus.

    python -m oracle.fit_cdf 0 1 2 3 4

Model: p_delta(x) = sigmoid(theta_delta - w.x), x = prefetch probabilities sorted descending,
theta_0 <= theta_1 <= ... kept ordered by theta_delta = theta_0 + cumulative softplus.  Full-batch
Adam in fp64, fixed iteration count, deterministic.
"""
from __future__ import annotations

import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import apex_oracle as ao  # noqa: E402
from paper_2608_11688_b200 import synth  # noqa: E402

N_CALIB = 2048
ITERS = 600


def calibration_set(cfg, layer):
    """x (sorted prefetch probabilities) and delta* of N_CALIB calibration tokens."""
    W_r, b_r, W_p, b_p = synth.router_weights(cfg, layer)
    h, hp = synth.hidden_states(cfg, layer, N_CALIB, 1, calib=True)
    Wp64, Wr64 = W_p.astype(np.float64), W_r.astype(np.float64)
    X = np.empty((N_CALIB, cfg.N))
    dstar = np.empty(N_CALIB, dtype=np.int64)
    # logits through the oracle's definitions (vectorised over tokens: same arithmetic, fp64 matmul)
    Zp = h[:, 0].astype(np.float64) @ Wp64.T + b_p.astype(np.float64)
    Zr = hp[:, 0].astype(np.float64) @ Wr64.T + b_r.astype(np.float64)
    for t in range(N_CALIB):
        q = ao.softmax(Zp[t])
        pi = ao.rank_desc(Zp[t])
        K_r = [int(e) for e in ao.rank_desc(Zr[t])[:cfg.k]]
        X[t] = q[pi]
        dstar[t] = ao.oracle_budget(pi, K_r, cfg.k)
    return X, dstar


def fit(X, dstar, N, k, iters=ITERS, lr=0.05):
    T = X.shape[0]
    nth = N - k + 1
    target = (np.arange(nth)[None, :] >= dstar[:, None]).astype(np.float64)     # I[delta >= delta*]
    w = np.zeros(N)
    # start from the empirical CDF of delta*
    cdf = np.clip(target.mean(0), 1e-3, 1 - 1e-3)
    th0 = np.log(cdf / (1 - cdf))
    t0 = th0[0]
    inc = np.maximum(np.diff(th0), 1e-3)
    u = np.log(np.expm1(inc))                                                    # softplus^-1
    params = np.concatenate([w, [t0], u])
    m = np.zeros_like(params); v = np.zeros_like(params)

    def unpack(p):
        w = p[:N]; t0 = p[N]; u = p[N + 1:]
        sp = np.logaddexp(0.0, u)
        theta = np.concatenate([[t0], t0 + np.cumsum(sp)])
        return w, theta, u

    for it in range(1, iters + 1):
        w, theta, u = unpack(params)
        s = X @ w
        z = theta[None, :] - s[:, None]
        p = 1.0 / (1.0 + np.exp(-z))
        g_z = (p - target) / T                                                   # d loss / d z
        g_w = -(g_z.sum(1)[:, None] * X).sum(0)
        g_theta = g_z.sum(0)
        # theta_j = t0 + sum_{i<=j} softplus(u_i): d/dt0 = sum_j, d/du_i = sigmoid(u_i) * sum_{j>=i+1}
        tail = np.cumsum(g_theta[::-1])[::-1]
        g_t0 = tail[0]
        g_u = (1.0 / (1.0 + np.exp(-u))) * tail[1:]
        g = np.concatenate([g_w, [g_t0], g_u])
        m = 0.9 * m + 0.1 * g; v = 0.999 * v + 0.001 * g * g
        params = params - lr * (m / (1 - 0.9 ** it)) / (np.sqrt(v / (1 - 0.999 ** it)) + 1e-8)
    w, theta, _ = unpack(params)
    return w.astype(np.float32), np.maximum.accumulate(theta.astype(np.float32))


def main(cfg_ids):
    out_dir = os.path.join(ROOT, "paper_2608_11688_b200", "data")
    os.makedirs(out_dir, exist_ok=True)
    for cid in cfg_ids:
        cfg = synth.CONFIGS[cid]
        W = np.zeros((cfg.L, cfg.N), np.float32)
        TH = np.zeros((cfg.L, cfg.N - cfg.k + 1), np.float32)
        cov = []
        for l in range(cfg.L):
            X, dstar = calibration_set(cfg, l)
            W[l], TH[l] = fit(X, dstar, cfg.N, cfg.k)
            # coverage at tau = 0.9 on the calibration set (sanity: should be near or above 0.9)
            t_tau = np.log(0.9 / 0.1)
            s = X @ W[l].astype(np.float64)
            ok = TH[l][None, :].astype(np.float64) - s[:, None] >= t_tau
            dhat = np.where(ok.any(1), ok.argmax(1), cfg.N - cfg.k)
            cov.append((float((dhat >= dstar).mean()), float(dhat.mean()), float(dstar.mean())))
        np.savez(os.path.join(out_dir, f"cdf_cfg{cid}.npz"), w=W, theta=TH)
        c = np.array(cov)
        print(f"config {cid}: coverage@0.9 mean {c[:,0].mean():.3f} min {c[:,0].min():.3f}; mean delta_hat {c[:,1].mean():.2f}; mean delta* {c[:,2].mean():.2f}")


if __name__ == "__main__":
    main([int(a) for a in sys.argv[1:]] or [0, 1, 2, 3, 4])
