"""GPU parity of apex_distill_router: the CUDA distillation of the prefetch router against the CPU one (oracle/distill.py)."""
import time

import numpy as np
import pytest
import torch

from paper_2608_11688_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


def _teacher(cfg, T):
    """Calibration tokens of a config: h (before attention), and the router's distribution on h' (after)."""
    W_r, b_r, W_p, b_p = synth.router_weights(cfg, 0)
    h, hp = synth.hidden_states(cfg, 0, T, 1, calib=True)
    H, Hp = h[:, 0].astype(np.float64), hp[:, 0].astype(np.float64)
    Z = Hp @ W_r.astype(np.float64).T + b_r.astype(np.float64)
    Z -= Z.max(1, keepdims=True)
    Qr = np.exp(Z)
    Qr /= Qr.sum(1, keepdims=True)
    return H.astype(np.float32), Qr.astype(np.float32), W_r, b_r, W_p, b_p


@pytest.mark.parametrize("shape", ["tiny", "config1"])
def test_distillation_matches_cpu(shape):
    from oracle import distill
    build.build()
    if shape == "tiny":
        cfg, T, iters = synth.tiny_config(d=96, N=9, k=2, I=16, C=4, sigma_p=0.5, cfg_id=295), 501, 60
    else:
        cfg, T, iters = synth.CONFIGS[1], 2048, 40
    H, Qr, W_r, b_r, W_p, b_p = _teacher(cfg, T)
    t0 = time.perf_counter()
    W_ref, b_ref = distill.distill(H, Qr, W_p, b_p, iters=iters, lr=0.01)
    t_cpu = time.perf_counter() - t0
    Hd, Qd = torch.from_numpy(H).cuda(), torch.from_numpy(Qr).cuda()
    binding.distill_router(Hd, Qd, W_p, b_p, iters=iters, lr=0.01)       # warm-up
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    W, b = binding.distill_router(Hd, Qd, W_p, b_p, iters=iters, lr=0.01)
    t_gpu = time.perf_counter() - t0
    # same iterations in fp64 on both sides (sums in another order); outputs are fp32
    assert np.abs(W - W_ref).max() <= 2e-6 * max(1.0, float(np.abs(W_ref).max())), np.abs(W - W_ref).max()
    assert np.abs(b - b_ref).max() <= 2e-6 * max(1.0, float(np.abs(b_ref).max())), np.abs(b - b_ref).max()
    W2, b2 = binding.distill_router(Hd, Qd, W_p, b_p, iters=iters, lr=0.01)
    assert np.array_equal(W, W2) and np.array_equal(b, b2)             # bit-reproducible
    l0, l1 = distill.kl_loss(H, Qr, W_p, b_p), distill.kl_loss(H, Qr, W, b)
    assert l1 < l0
    print(f"distill {shape}: T={T} N={cfg.N} d={cfg.d} iters={iters}  gpu {t_gpu*1e3:.1f} ms  cpu {t_cpu*1e3:.1f} ms  "
          f"KL {l0:.4f} -> {l1:.4f}  max|dW| {np.abs(W - W_ref).max():.2e}")


def test_distillation_rejects_bad_arguments():
    build.build()
    H = torch.zeros((8, 16), dtype=torch.float32, device="cuda")
    Q = torch.zeros((8, 70), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.ApexError):
        binding.distill_router(H, Q, np.zeros((70, 16), np.float32), np.zeros(70, np.float32))      # N > 64
