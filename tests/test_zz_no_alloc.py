"""The allocation-free gate entry point against the context API.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has
already run every other test.  apex_route_topk_static serves callers that cannot allocate device
memory (a fixed memory pool owns the GPU); it must give what apex_route_topk gives, on repeated
calls that share its built-in scratch array."""
import numpy as np
import pytest
import torch

from paper_2608_11688_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


def _context_gate(cfg, W_r, b_r, hp, B):
    a = binding.Apex(d=cfg.d, N=cfg.N, k=cfg.k, I=cfg.I, C_slots=cfg.C, max_batch=B)
    try:
        a.set_router(0, W_r, b_r)
        idx = torch.empty((B, cfg.k), dtype=torch.int32, device="cuda")
        alpha = torch.empty((B, cfg.N), dtype=torch.float32, device="cuda")
        a.route_topk(0, hp, B, idx, alpha)
        torch.cuda.synchronize()
        return idx.cpu().numpy().copy(), alpha.cpu().numpy().copy()
    finally:
        a.destroy()


def test_static_gate_matches_context_gate_on_two_calls_in_a_row():
    build.build()
    cfg = synth.tiny_config(d=1536, N=40, k=8, I=16, C=20, T=4, zipf_s=1.1, cfg_id=950)
    W_r, b_r, _, _ = synth.router_weights(cfg, 0)
    W_dev = torch.from_numpy(W_r).cuda()
    b_dev = torch.from_numpy(b_r).cuda()
    h5, hp5 = synth.hidden_states(cfg, 0, 2, B=5)
    h1, hp1 = synth.hidden_states(cfg, 0, 2, B=1)
    free_before = torch.cuda.mem_get_info()[0]
    # two calls in a row with different shapes: the second must not see anything of the first
    for call, hp in enumerate([hp5[0], hp1[1], hp5[1]]):
        B = hp.shape[0]
        hp_dev = torch.from_numpy(hp).cuda()
        idx = torch.full((B, cfg.k), -1, dtype=torch.int32, device="cuda")
        alpha = torch.zeros((B, cfg.N), dtype=torch.float32, device="cuda")
        binding.route_topk_static(W_dev, b_dev, hp_dev, cfg.k, idx, alpha)
        torch.cuda.synchronize()
        ref_idx, ref_alpha = _context_gate(cfg, W_r, b_r, hp_dev, B)
        np.testing.assert_array_equal(idx.cpu().numpy(), ref_idx)                     # indices: bit-exact
        np.testing.assert_allclose(alpha.cpu().numpy(), ref_alpha, atol=1e-6, rtol=1e-5)
        assert abs(float(alpha.sum()) - B) < 1e-4
    assert torch.cuda.mem_get_info()[0] <= free_before + (64 << 20)


def test_static_gate_refuses_sizes_beyond_its_scratch():
    build.build()
    W = torch.zeros((8, 256), device="cuda")
    hp = torch.zeros((65, 256), device="cuda")          # B = 65 > 64
    idx = torch.zeros((65, 2), dtype=torch.int32, device="cuda")
    alpha = torch.zeros((65, 8), device="cuda")
    with pytest.raises(binding.ApexError) as ei:
        binding.route_topk_static(W, None, hp, 2, idx, alpha)
    assert ei.value.code == binding.APEX_EINVAL and "scratch" in str(ei.value)
    with pytest.raises(binding.ApexError) as ei:
        binding.route_topk_static(torch.zeros((8, 258), device="cuda"), None, torch.zeros((1, 258), device="cuda"), 2,
                                  idx[:1].contiguous(), alpha[:1].contiguous())
    assert ei.value.code == binding.APEX_EINVAL
