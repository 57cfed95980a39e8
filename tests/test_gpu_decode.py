"""GPU parity of the whole-token call (apex_decode_token): at B = 1 one persistent kernel over all layers, against
the CPU oracle layer by layer, and against the per-layer kernel sequence it replaces."""
import numpy as np
import pytest
import torch

from paper_2608_11688_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _harness():
    import harness
    return harness


def _decode(cfg, *, mode, tau, T, B=1, layers=None, C=None, norm_topk=1, cache_reuse=1, flags=0, prob=None, cdf="handset",
            layers_checked=None, ffn_token_stride=1, max_near_ties=0, host_buffers=False, check_counters=True):
    hz = _harness()
    prob = prob or hz.Problem(cfg, layers=layers, cdf=cdf)
    apex = prob.make_ctx(C=C, max_batch=B, norm_topk=norm_topk, cache_reuse=cache_reuse, flags=flags)
    try:
        n0 = apex.launch_count()
        rep = hz.run_decode_lockstep(prob, apex, mode=mode, tau=tau, T=T, B=B, C=C, norm_topk=bool(norm_topk),
                                     cache_reuse=bool(cache_reuse), layers_checked=layers_checked,
                                     ffn_token_stride=ffn_token_stride, max_near_ties=max_near_ties, host_buffers=host_buffers)
        stats = apex.get_stats()
        launches = apex.launch_count() - n0
    finally:
        apex.destroy()
    assert stats["timeouts"] == 0
    if check_counters and rep.near_ties == 0 and layers_checked is None:
        keys = ["hits_R", "prefetch_copies", "demand_copies", "substitutions"]
        if not (tau < 0):
            keys += ["sum_delta_hat", "sum_delta_star", "sum_ncand", "hits_P", "covered", "capped"]
        ours = {"prefetch_copies": rep.n_prefetch_copies, "demand_copies": rep.n_demand_copies, "substitutions": rep.n_subst}
        for key in keys:
            assert stats[key] == ours.get(key, getattr(rep, key, None)), (key, stats[key], ours.get(key, getattr(rep, key, None)))
    return rep, stats, launches


@pytest.mark.parametrize("mode", ["exact", "stall_free"])
@pytest.mark.parametrize("d,N,k,I,C,L,Ish", [(256, 8, 2, 24, 4, 3, 0), (512, 12, 3, 40, 6, 2, 16), (768, 33, 5, 17, 9, 4, 0),
                                             (1024, 64, 8, 16, 16, 2, 0), (1536, 40, 8, 64, 20, 5, 0), (2048, 60, 4, 32, 30, 3, 48),
                                             (3072, 5, 1, 9, 2, 2, 0), (4096, 8, 2, 24, 4, 3, 0)])
def test_persistent_token_kernel_tiny_shapes(d, N, k, I, C, L, Ish, mode):
    cfg = synth.tiny_config(d=d, N=N, k=k, I=I, C=C, L=L, T=6, I_shared=Ish, sigma_p=1.0, cfg_id=400 + N)
    rep, stats, launches = _decode(cfg, mode=mode, tau=0.7, T=6)
    assert rep.layer_steps == 6 * L and rep.ffn_checked == 6 * L
    assert launches == 6 or not _harness().token_kernel_expected()       # one kernel per token
    assert stats["tokens"] == 6 * L and stats["routed"] == 6 * L * k
    if mode == "stall_free":
        assert rep.n_demand_copies == 0


@pytest.mark.parametrize("mode", ["exact", "stall_free"])
def test_persistent_token_kernel_with_a_gated_shared_expert(mode):
    cfg = synth.tiny_config(d=1024, N=24, k=6, I=96, C=12, L=4, T=5, I_shared=64, sigma_p=1.0, cfg_id=414)
    prob = _harness().Problem(cfg, gated_shared=True)
    rep, stats, launches = _decode(cfg, mode=mode, tau=0.8, T=5, prob=prob)
    assert rep.near_ties == 0 and rep.ffn_checked == 5 * 4
    assert launches == 5 or not _harness().token_kernel_expected()     # one launch per token


@pytest.mark.parametrize("mode", ["exact", "stall_free"])
@pytest.mark.parametrize("fmt", ["fp8", "fp4"])
@pytest.mark.parametrize("d,N,k,I,C,L,Ish", [(512, 12, 3, 40, 6, 3, 16), (1024, 64, 8, 16, 16, 2, 0), (1536, 40, 8, 64, 20, 4, 0),
                                             (2048, 60, 4, 32, 30, 3, 48), (4096, 8, 2, 24, 4, 3, 0)])
def test_persistent_token_kernel_quantised_stores(d, N, k, I, C, L, Ish, fmt, mode):
    # the token kernel on e4m3 / e2m1 expert stores: rows shorter than a vector of y (the cross-warp reduction then
    # uses the start of the ring), more and smaller ring stages, the same decisions
    cfg = synth.tiny_config(d=d, N=N, k=k, I=I, C=C, L=L, T=5, I_shared=Ish, sigma_p=1.0, cfg_id=420 + N)
    prob = _harness().Problem(cfg, fp8=(fmt == "fp8"), fp4=(fmt == "fp4"))
    rep, stats, launches = _decode(cfg, mode=mode, tau=0.7, T=5, prob=prob)
    assert rep.layer_steps == 5 * L and rep.ffn_checked == 5 * L and rep.near_ties == 0
    assert launches == 5 or not _harness().token_kernel_expected()       # one kernel per token: the persistent path ran


@pytest.mark.parametrize("tau", [-1.0, 0.0, 0.97, 1.0])
def test_persistent_token_kernel_policies_and_budget_extremes(tau):
    cfg = synth.tiny_config(d=512, N=16, k=4, I=32, C=8, L=3, T=8, sigma_p=0.8, cfg_id=410)
    rep, stats, _ = _decode(cfg, mode="exact", tau=tau, T=8)
    if tau < 0:
        assert stats["prefetch_copies"] == 0 and stats["demand_copies"] > 0
    if tau == 1.0:
        assert stats["capped"] == 8 * 3


def test_persistent_token_kernel_minimal_cache_staging_policy_and_plain_gates():
    cfg = synth.tiny_config(d=256, N=10, k=3, I=16, C=3, L=2, T=12, sigma_p=1.5, cfg_id=411)
    rep, stats, _ = _decode(cfg, mode="exact", tau=0.9, T=12)
    assert rep.n_miss_steps > 0 and stats["demand_copies"] == rep.n_demand_copies > 0     # waited for inside the kernel
    rep, stats, _ = _decode(cfg, mode="stall_free", tau=0.9, T=12)
    assert rep.n_subst > 0
    cfg = synth.tiny_config(d=512, N=12, k=3, I=24, C=7, L=2, T=8, sigma_p=1.0, cfg_id=412)
    rep, stats, _ = _decode(cfg, mode="stall_free", tau=0.8, T=8, cache_reuse=0)           # load-use-evict per layer-step
    assert stats["prefetch_copies"] == stats["sum_ncand"]
    _decode(cfg, mode="exact", tau=0.8, T=6, norm_topk=0)


def test_persistent_kernel_equals_the_per_layer_sequence_and_host_buffer_variant():
    cfg = synth.tiny_config(d=1024, N=24, k=6, I=96, C=12, L=4, T=6, I_shared=32, sigma_p=1.0, cfg_id=413)
    hz = _harness()
    prob = hz.Problem(cfg)
    hs = [synth.hidden_states(cfg, l, cfg.T, 1) for l in range(cfg.L)]
    h = torch.from_numpy(np.stack([x[0] for x in hs], 1)).cuda()
    hp = torch.from_numpy(np.stack([x[1] for x in hs], 1)).cuda()
    outs = []
    for flags in (0, binding.FLAG_LAYER_LAUNCHES):
        apex = prob.make_ctx(flags=flags)
        try:
            y = torch.zeros((cfg.T, cfg.L, 1, cfg.d), dtype=torch.float32, device="cuda")
            n0 = apex.launch_count()
            for t in range(cfg.T):
                apex.decode_token(h[t], hp[t], 1, 0.8, "exact", y[t])
            torch.cuda.synchronize()
            n_launch = apex.launch_count() - n0
            st = apex.get_stats()
            keep = {k_: st[k_] for k_ in ("tokens", "routed", "hits_P", "hits_R", "covered", "prefetch_copies", "demand_copies",
                                          "sum_delta_hat", "sum_delta_star", "sum_ncand", "capped", "substitutions", "timeouts",
                                          "bytes_copied", "layer_steps")}
            outs.append((y.cpu().numpy(), keep, [apex.get_slot_table(l) for l in range(cfg.L)], n_launch))
        finally:
            apex.destroy()
    assert outs[0][1] == outs[1][1] and outs[0][1]["timeouts"] == 0
    assert (outs[0][3] == cfg.T or not hz.token_kernel_expected()) and outs[1][3] >= 4 * cfg.L * cfg.T
    for t0, t1 in zip(outs[0][2], outs[1][2]):
        assert list(t0[0]) == list(t1[0]) and list(t0[1]) == list(t1[1]) and t0[2] == t1[2]
    np.testing.assert_allclose(outs[0][0], outs[1][0], rtol=0, atol=2e-6 * float(np.abs(outs[1][0]).max()))
    # pinned host buffers in, y out, through the same kernel
    _decode(cfg, mode="stall_free", tau=0.8, T=3, prob=prob, host_buffers=True)


def test_persistent_kernel_without_the_attention_standin():
    cfg = synth.tiny_config(d=512, N=12, k=3, I=40, C=6, L=3, T=5, sigma_p=1.0, cfg_id=414)
    _decode(cfg, mode="exact", tau=0.7, T=5, flags=binding.FLAG_SKIP_STANDIN)


def test_persistent_kernel_wait_runs_out_and_the_context_recovers():
    if not _harness().token_kernel_expected():
        pytest.skip("launch calls may block here: apex_decode_token keeps to per-layer launches")
    # a slot-ready flag is withheld (host-side hook): the kernel's bounded wait runs out, every CTA leaves, the call
    # reports APEX_ETIMEOUT; afterwards the context decodes again (per-layer launches with host-side miss correction)
    cfg = synth.tiny_config(d=256, N=8, k=4, I=16, C=8, L=2, T=8, sigma_p=0.0, cfg_id=415)
    hz = _harness()
    prob = hz.Problem(cfg)
    a = prob.make_ctx(wait_limit_ns=50_000_000)
    try:
        hs = [synth.hidden_states(cfg, l, cfg.T, 1) for l in range(cfg.L)]
        h = torch.from_numpy(np.stack([x[0] for x in hs], 1)).cuda()
        hp = torch.from_numpy(np.stack([x[1] for x in hs], 1)).cuda()
        y = torch.zeros((cfg.L, 1, cfg.d), device="cuda")
        a.test_inject(2)          # the flag of the first copy (the expert the prefetch router ranks first) is never written
        raised_at = None
        for t in range(6):        # whoever executes that expert waits in vain
            try:
                a.decode_token(h[t], hp[t], 1, 1.0, "stall_free", y)
                torch.cuda.synchronize()
            except binding.ApexError as e:
                assert e.code == binding.APEX_ETIMEOUT
                raised_at = t
                break
        torch.cuda.synchronize()
        assert raised_at is not None and a.get_stats()["timeouts"] > 0
        for t in range(6, 8):
            try:
                a.decode_token(h[t], hp[t], 1, 0.9, "exact", y)
            except binding.ApexError as e:
                assert e.code == binding.APEX_ETIMEOUT            # reported once more at most
                a.decode_token(h[t], hp[t], 1, 0.9, "exact", y)
            torch.cuda.synchronize()
            assert torch.isfinite(y).all()
    finally:
        a.destroy()


# ------------------------------------------------------------------ the paper-shaped configs at their full size
def _sampled(step, L):
    """Layers replayed by the oracle for token t: every `step`-th, the offset moving with t, plus the last layer."""
    return lambda t: sorted(set(list(range((t * 3) % step, L, step)) + [L - 1]))


@pytest.mark.parametrize("mode", ["exact", "stall_free"])
def test_config2_full_size_all_layers_sampled(mode):
    """Config 2 (OLMoE shape: 16 layers, 64 experts of 12 MiB, Zipf router bias, 24 slots, fitted confidence model)
    through the whole-token call.  Slot tables of every layer before and after each token; sampled layers replayed by
    the oracle: copy lists and tables bit-exact, y by tolerance."""
    cfg = synth.CONFIGS[2]
    rep, stats, launches = _decode(cfg, mode=mode, tau=0.9, T=3, cdf="fitted", layers_checked=_sampled(5, cfg.L))
    assert rep.ffn_checked >= 9 and stats["tokens"] == 3 * cfg.L
    assert launches == 3 or not _harness().token_kernel_expected()
    print("config2 full", mode, rep)


@pytest.mark.parametrize("B,stride,T", [(1, 1, 2), (32, 8, 1), (256, 64, 1)])
def test_config4_full_size_all_layers_sampled(B, stride, T):
    """Config 4 (Qwen1.5-MoE shape: 24 layers, 60 experts of 16.5 MiB, shared expert, 30 slots), exact mode: B = 1 on
    the persistent kernel, B = 32 and 256 on the tensor-core grouped GEMMs, where the distinct routed experts of a step
    exceed the 30 slots and the step runs in waves."""
    cfg = synth.CONFIGS[4]
    rep, stats, launches = _decode(cfg, mode="exact", tau=0.9, T=T, B=B, cdf="fitted", layers_checked=_sampled(9, cfg.L),
                                   ffn_token_stride=stride)
    assert stats["tokens"] == T * B * cfg.L and rep.ffn_checked >= 3 * max(1, B // stride)
    if B >= 32:
        assert stats["extra_waves"] > 0
    print("config4 full", B, rep, {k_: stats[k_] for k_ in ("extra_waves", "demand_copies", "prefetch_copies")})


def test_config4_shape_stall_free_on_the_tensor_core_path():
    cfg = synth.CONFIGS[4]
    hz = _harness()
    prob = hz.Problem(cfg, layers=2, cdf="fitted")
    for B, stride in ((32, 8), (128, 32)):
        rep, stats, _ = _decode(cfg, mode="stall_free", tau=0.9, T=2, B=B, prob=prob, ffn_token_stride=stride)
        assert stats["demand_copies"] == 0 and stats["substitutions"] == rep.n_subst > 0
        print("config4 stall-free tc", B, rep)


def _host_memory_available_gib():
    try:
        for ln in open("/proc/meminfo"):
            if ln.startswith("MemAvailable:"):
                return int(ln.split()[1]) / (1 << 20)
    except OSError:
        pass
    return 0.0


def test_config3_all_layers():
    """Config 3 (Mixtral-8x7B shape: 32 layers, 8 experts of 336 MiB, 4 slots, prefetch noise 0.5): all 32 layers through
    the whole-token call, both modes.  The full expert store is 84 GiB of pinned host memory; it is allocated only if
    the host reports at least 1.5 times that as available, otherwise eight physical layer stores are aliased onto the
    32 layers (routers, confidence models and hidden states stay per layer)."""
    cfg = synth.CONFIGS[3]
    hz = _harness()
    need_gib = cfg.L * cfg.N * cfg.expert_bytes / (1 << 30)
    avail = _host_memory_available_gib()
    full = avail >= 1.5 * need_gib
    prob = None
    if full:
        try:
            prob = hz.Problem(cfg, cdf="fitted")
        except RuntimeError as e:            # pinning refused: fall back
            print("config3: full pinned store refused:", str(e)[:200])
            full = False
    if prob is None:
        prob = hz.Problem(cfg, cdf="fitted", store_layers=8)
    print(f"config3: host MemAvailable {avail:.0f} GiB, store {need_gib:.0f} GiB -> {'full store' if full else '8 physical layer stores, aliased'}")
    for mode in ("exact", "stall_free"):
        rep, stats, launches = _decode(cfg, mode=mode, tau=0.9, T=2, prob=prob, layers_checked=_sampled(11, cfg.L))
        assert stats["tokens"] == 2 * cfg.L and rep.ffn_checked >= 6
        assert launches == 2 or not _harness().token_kernel_expected()
        print("config3 all layers", mode, rep)


@pytest.mark.parametrize("delta", [0, 4, 8])
def test_static_budget_baselines_against_the_oracle(delta):
    """The static top-k / top-(k + delta) prefetch baselines of Sec. V-A (same ranking, fixed budget: w = 0 and a step
    in theta): every decision against the oracle under that model, per call and through the whole-token kernel."""
    cfg = synth.tiny_config(d=512, N=24, k=4, I=32, C=16, L=2, T=8, sigma_p=1.0, cfg_id=416)
    hz = _harness()
    prob = hz.Problem(cfg, cdf=("static", delta))
    apex = prob.make_ctx()
    try:
        rep = hz.run_lockstep(prob, apex, mode="exact", tau=0.9, T=cfg.T)
        st = apex.get_stats()
    finally:
        apex.destroy()
    assert st["sum_delta_hat"] == delta * cfg.T * cfg.L == rep.sum_delta_hat and st["sum_ncand"] == (cfg.k + delta) * cfg.T * cfg.L
    rep, stats, _ = _decode(cfg, mode="stall_free", tau=0.9, T=cfg.T, prob=prob)
    assert stats["sum_delta_hat"] == delta * cfg.T * cfg.L
