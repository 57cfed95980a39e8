"""The allocation-free gate entry point against the context API and the CPU oracle.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has
already run every other test.  apex_route_topk_static serves callers that cannot allocate device
memory (a fixed memory pool owns the GPU); it must give what apex_route_topk gives, on repeated
calls that share its built-in scratch array, and it must really allocate nothing."""
import numpy as np
import pytest
import torch

from oracle import apex_oracle as ao
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


def _check_against_oracle(W_r, b_r, hp, k, idx, alpha):
    """Indices bit-exact and alpha to 1e-6 against the fp64 oracle; a token may differ only where the oracle's own
    deciding logit gap is below the near-tie tolerance.  Returns the number of such tokens."""
    near = 0
    for b in range(hp.shape[0]):
        z_r, K_r, a_ref = ao.route_topk(W_r, b_r, hp[b], k)
        np.testing.assert_allclose(alpha[b], a_ref, atol=1e-6, rtol=1e-5)
        if list(idx[b]) != K_r:
            assert ao.min_adjacent_gap(z_r, upto=k) < ao.NEAR_TIE_LOGIT, (b, list(idx[b]), K_r)
            near += 1
    return near


def test_static_gate_matches_context_gate_and_oracle_on_two_calls_in_a_row():
    build.build()
    cfg = synth.tiny_config(d=1536, N=40, k=8, I=16, C=20, T=4, zipf_s=1.1, cfg_id=950)
    W_r, b_r, _, _ = synth.router_weights(cfg, 0)
    W_dev = torch.from_numpy(W_r).cuda()
    b_dev = torch.from_numpy(b_r).cuda()
    h5, hp5 = synth.hidden_states(cfg, 0, 2, B=5)
    h1, hp1 = synth.hidden_states(cfg, 0, 2, B=1)
    near = 0
    # calls in a row with different shapes: a call must not see anything of the one before it
    for call, hp in enumerate([hp5[0], hp1[1], hp5[1]]):
        B = hp.shape[0]
        hp_dev = torch.from_numpy(hp).cuda()
        idx = torch.full((B, cfg.k), -1, dtype=torch.int32, device="cuda")
        alpha = torch.zeros((B, cfg.N), dtype=torch.float32, device="cuda")
        binding.route_topk_static(W_dev, b_dev, hp_dev, cfg.k, idx, alpha)
        torch.cuda.synchronize()
        ref_idx, ref_alpha = _context_gate(cfg, W_r, b_r, hp_dev, B)
        np.testing.assert_array_equal(idx.cpu().numpy(), ref_idx)                     # the existing entry point: bit-exact
        np.testing.assert_allclose(alpha.cpu().numpy(), ref_alpha, atol=1e-6, rtol=1e-5)
        assert abs(float(alpha.sum()) - B) < 1e-4
        near += _check_against_oracle(W_r, b_r, hp, cfg.k, idx.cpu().numpy(), alpha.cpu().numpy())
    assert near == 0


def test_static_gate_at_the_edge_of_its_scratch_and_with_a_ragged_last_group():
    # B = 64 tokens of N = 64 experts fill the built-in array exactly; B = 63 leaves the last token group partial
    build.build()
    cfg = synth.tiny_config(d=512, N=64, k=16, I=16, C=32, T=2, cfg_id=951)
    W_r, b_r, _, _ = synth.router_weights(cfg, 0)
    W_dev, b_dev = torch.from_numpy(W_r).cuda(), torch.from_numpy(b_r).cuda()
    near = 0
    for t, B in enumerate([64, 63]):
        _, hp = synth.hidden_states(cfg, 0, 2, B=B)
        hp_dev = torch.from_numpy(hp[t]).cuda()
        idx = torch.full((B, cfg.k), -1, dtype=torch.int32, device="cuda")
        alpha = torch.zeros((B, cfg.N), dtype=torch.float32, device="cuda")
        binding.route_topk_static(W_dev, b_dev, hp_dev, cfg.k, idx, alpha)
        torch.cuda.synchronize()
        ref_idx, ref_alpha = _context_gate(cfg, W_r, b_r, hp_dev, B)
        np.testing.assert_array_equal(idx.cpu().numpy(), ref_idx)
        np.testing.assert_allclose(alpha.cpu().numpy(), ref_alpha, atol=1e-6, rtol=1e-5)
        near += _check_against_oracle(W_r, b_r, hp[t], cfg.k, idx.cpu().numpy(), alpha.cpu().numpy())
    assert near == 0


@pytest.mark.parametrize("d", [260, 4, 1000])
def test_static_gate_accepts_widths_the_context_api_does_not(d):
    # the context API wants d in multiples of 256; this entry point takes any multiple of 4: checked against the oracle
    build.build()
    rng = np.random.default_rng(952 + d)
    N, k = 12, 3
    W_r = (rng.standard_normal((N, d)) / np.sqrt(d)).astype(np.float32)
    b_r = (0.1 * rng.standard_normal(N)).astype(np.float32)
    near = 0
    for B in (1, 7):
        hp = synth.round_to_bf16_values(rng.standard_normal((B, d)).astype(np.float32))
        idx = torch.full((B, k), -1, dtype=torch.int32, device="cuda")
        alpha = torch.zeros((B, N), dtype=torch.float32, device="cuda")
        binding.route_topk_static(torch.from_numpy(W_r).cuda(), torch.from_numpy(b_r).cuda(), torch.from_numpy(hp).cuda(), k, idx, alpha)
        torch.cuda.synchronize()
        near += _check_against_oracle(W_r, b_r, hp, k, idx.cpu().numpy(), alpha.cpu().numpy())
    assert near == 0


def test_static_gate_allocates_nothing():
    """Free device memory, read right before and right after a burst of calls, must not drop, and torch's own
    allocator must not have been asked for anything.  Everything the calls touch is allocated beforehand, and one
    call per kernel variant has already run (loading a kernel's code for the first time takes device memory once,
    like loading the library does; the entry point's promise is about its calls)."""
    build.build()
    cfg = synth.tiny_config(d=1024, N=64, k=16, I=16, C=32, T=1, cfg_id=953)
    W_r, b_r, _, _ = synth.router_weights(cfg, 0)
    W_dev, b_dev = torch.from_numpy(W_r).cuda(), torch.from_numpy(b_r).cuda()
    cases = []
    for B in (1, 5, 64):
        _, hp = synth.hidden_states(cfg, 0, 1, B=B)
        cases.append((torch.from_numpy(hp[0]).cuda(), torch.empty((B, cfg.k), dtype=torch.int32, device="cuda"),
                      torch.empty((B, cfg.N), dtype=torch.float32, device="cuda")))
    for hp_dev, idx, alpha in cases:                                  # first use of each kernel variant
        binding.route_topk_static(W_dev, b_dev, hp_dev, cfg.k, idx, alpha)
    torch.cuda.synchronize()
    torch_before = torch.cuda.memory_allocated()
    reserved_before = torch.cuda.memory_reserved()
    free0 = torch.cuda.mem_get_info()[0]
    for rep in range(8):
        for hp_dev, idx, alpha in cases:
            binding.route_topk_static(W_dev, b_dev, hp_dev, cfg.k, idx, alpha)
    torch.cuda.synchronize()
    free1 = torch.cuda.mem_get_info()[0]
    assert free1 >= free0, f"device memory dropped by {free0 - free1} bytes across the calls"
    assert torch.cuda.memory_allocated() == torch_before and torch.cuda.memory_reserved() == reserved_before


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
