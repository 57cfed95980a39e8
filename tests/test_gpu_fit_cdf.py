"""GPU parity of apex_fit_cdf: the CUDA fit of the confidence model against the CPU fit (oracle/fit_cdf.py)."""
import time

import numpy as np
import pytest
import torch

from paper_2608_11688_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


def _calibration(cfg, layer):
    from oracle import fit_cdf
    return fit_cdf.calibration_set(cfg, layer)


@pytest.mark.parametrize("shape", ["tiny", "config1", "config2"])
def test_fit_matches_cpu_fit(shape):
    from oracle import fit_cdf
    build.build()
    if shape == "tiny":
        cfg, iters = synth.tiny_config(d=256, N=12, k=3, I=16, C=6, sigma_p=0.6, cfg_id=290), 150
    else:
        cfg, iters = synth.CONFIGS[1 if shape == "config1" else 2], 600
    X, dstar = _calibration(cfg, 0)
    if shape == "tiny":                      # a ragged token count: not a multiple of the CTA's chunk
        X, dstar = X[:1000], dstar[:1000]
    t0 = time.perf_counter()
    w_ref, th_ref = fit_cdf.fit(X, dstar, cfg.N, cfg.k, iters=iters)
    t_cpu = time.perf_counter() - t0
    Xd = torch.from_numpy(X).cuda()
    dd = torch.from_numpy(dstar.astype(np.int32)).cuda()
    binding.fit_cdf(Xd, dd, cfg.k, iters=iters)          # warm-up (module load, graph instantiation)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    w, th = binding.fit_cdf(Xd, dd, cfg.k, iters=iters)
    t_gpu = time.perf_counter() - t0
    # Both sides run the same iterations in fp64; they differ in the order of the sums and in exp() to an ulp,
    # which Adam carries along without amplifying much.  The outputs are fp32: allow a few fp32 ulps.
    scale_w, scale_t = float(np.abs(w_ref).max()), float(np.abs(th_ref).max())
    assert np.abs(w - w_ref).max() <= 1e-5 * max(scale_w, 1.0), np.abs(w - w_ref).max()
    assert np.abs(th - th_ref).max() <= 1e-5 * max(scale_t, 1.0), np.abs(th - th_ref).max()
    assert np.all(np.diff(th) >= 0)
    # the budgets the two models choose on the calibration set are the same (threshold margins permitting)
    t_tau = np.log(0.9 / 0.1)

    def budgets(w_, th_):
        s = X @ w_.astype(np.float64)
        marg = th_[None, :].astype(np.float64) - s[:, None] - t_tau
        ok = marg >= 0
        return np.where(ok.any(1), ok.argmax(1), cfg.N - cfg.k), np.abs(marg).min(1)
    d_gpu, _ = budgets(w, th)
    d_ref, margin = budgets(w_ref, th_ref)
    differs = d_gpu != d_ref
    assert np.all(margin[differs] < 1e-4), int(differs.sum())
    # bit-reproducible
    w2, th2 = binding.fit_cdf(Xd, dd, cfg.k, iters=iters)
    assert np.array_equal(w, w2) and np.array_equal(th, th2)
    print(f"fit_cdf {shape}: T={len(dstar)} N={cfg.N} iters={iters}  gpu {t_gpu*1e3:.1f} ms  cpu {t_cpu*1e3:.1f} ms  "
          f"max|dw| {np.abs(w - w_ref).max():.2e} max|dtheta| {np.abs(th - th_ref).max():.2e}")


def test_fit_rejects_bad_arguments():
    build.build()
    X = torch.zeros((8, 70), dtype=torch.float64, device="cuda")
    d = torch.zeros((8,), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.ApexError):
        binding.fit_cdf(X, d, 4)                       # N > 64
    with pytest.raises(binding.ApexError):
        binding.fit_cdf(X[:, :16].contiguous(), d, 17)  # k > N
