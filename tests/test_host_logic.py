"""CPU-only tests of the library's host side: the shared object loads and exports every symbol the
header declares, the C++ slot planner agrees with the oracle's slot cache decision by decision,
and the host helpers behave.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

from oracle import apex_oracle as ao
from paper_2608_11688_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "apex.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(apex_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_symbols()
    assert len(names) >= 30
    for n in names:
        assert hasattr(lib, n), n
        assert n in binding.SIGNATURES, f"{n} declared in apex.h but not bound"
    assert sorted(binding.SIGNATURES) == names


def test_null_and_bad_arguments_are_rejected_without_cuda(lib):
    assert lib.apex_destroy(None) == binding.APEX_EINVAL
    assert lib.apex_create(None, None) == binding.APEX_EINVAL
    cfg = binding.ApexConfig(d=1000, N=8, k=2, I=8, I_shared=0, C=4, L=1, max_batch=1, norm_topk=1, cache_reuse=1)
    h = ctypes.c_void_p()
    assert lib.apex_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.APEX_EINVAL   # d not supported
    for bad in (dict(N=65), dict(k=0), dict(C=1), dict(C=9), dict(max_batch=257), dict(L=0)):
        kw = dict(d=256, N=8, k=2, I=8, I_shared=0, C=4, L=1, max_batch=1, norm_topk=1, cache_reuse=1)
        kw.update(bad)
        cfg = binding.ApexConfig(**kw)
        assert lib.apex_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.APEX_EINVAL, bad
    # the e4m3 store needs one of the widths its kernel was built for
    cfg = binding.ApexConfig(d=768, N=8, k=2, I=8, I_shared=0, C=4, L=1, max_batch=1, norm_topk=1, cache_reuse=1,
                             flags=binding.FLAG_FP8_EXPERTS)
    assert lib.apex_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.APEX_EINVAL
    cfg = binding.ApexConfig(d=512, N=8, k=2, I=8, I_shared=0, C=4, L=1, max_batch=1, norm_topk=1, cache_reuse=1,
                             flags=binding.FLAG_FP8_EXPERTS | binding.FLAG_FP4_EXPERTS)
    assert lib.apex_create(ctypes.byref(cfg), ctypes.byref(h)) == binding.APEX_EINVAL   # one format at a time
    assert lib.apex_slots_create(8, 9, 1) is None
    assert lib.apex_launch_count(None) == -1


def test_fp4_store_generator_round_trips_within_e2m1_precision():
    import numpy as np
    import torch
    from paper_2608_11688_b200 import synth
    cfg = synth.tiny_config(d=512, N=3, k=1, I=5)
    w = synth.expert_store(cfg, 0).to(torch.float32).numpy()
    q = synth.expert_store_fp4(cfg, 0)
    assert q.shape == (3, 5, synth.fp4_row_bytes(512)) and synth.fp4_row_bytes(512) % 16 == 0
    dq = synth.dequantize_store_fp4(q, 512)
    # a block's scale is the smallest power of two that maps its maximum into [-6, 6]; the widest gap between
    # neighbouring e2m1 values there is 2 (between 4 and 6), so the error is at most one scale unit, and the
    # scale is below amax / 3
    blk_w = w.reshape(3, 5, 3, 16, 32)
    blk_e = np.abs(dq - w).reshape(3, 5, 3, 16, 32)
    amax = np.abs(blk_w).max(-1, keepdims=True)
    assert np.all(blk_e <= amax / 3 + 1e-12)
    # quantising what was dequantised reproduces the same values (a block may be re-coded with a smaller scale)
    q2 = synth.quantize_store_fp4(torch.from_numpy(dq.astype(np.float32)))
    assert np.array_equal(synth.dequantize_store_fp4(q2, 512), dq)


def test_fp8_store_generator_round_trips_within_e4m3_precision():
    import numpy as np
    import torch
    from paper_2608_11688_b200 import synth
    cfg = synth.tiny_config(d=512, N=3, k=1, I=5)
    w = synth.expert_store(cfg, 0).to(torch.float32).numpy()
    q = synth.expert_store_fp8(cfg, 0)
    assert q.shape == (3, 5, 3 * 512 + 16) and q.dtype == torch.uint8
    dq = synth.dequantize_store_fp8(q, 512)
    # e4m3 keeps 3 mantissa bits: relative error <= 2^-4 for normal codes; the per-row scale maps the
    # row maximum to 448, so nothing overflows and the absolute error is <= amax * 2^-4
    amax = np.abs(w).max(axis=-1, keepdims=True)
    assert np.all(np.abs(dq - w) <= amax / 16 + 1e-12)
    assert np.all(q[..., 3 * 512 + 12:].numpy() == 0)                          # padding bytes
    # the row maximum is reproduced exactly (code 448 times scale)
    assert np.allclose(np.abs(dq).max(axis=-1, keepdims=True), amax, rtol=1e-6)


def test_pack_expert_transposes_down(lib):
    d, I = 8, 3
    rng = np.random.default_rng(0)
    gate = rng.integers(0, 2 ** 16, (I, d)).astype(np.uint16)
    up = rng.integers(0, 2 ** 16, (I, d)).astype(np.uint16)
    down = rng.integers(0, 2 ** 16, (d, I)).astype(np.uint16)
    out = np.zeros((I, 3, d), np.uint16)
    assert lib.apex_pack_expert(gate.ctypes.data, up.ctypes.data, down.ctypes.data, d, I, out.ctypes.data) == 0
    np.testing.assert_array_equal(out[:, 0], gate)
    np.testing.assert_array_equal(out[:, 1], up)
    np.testing.assert_array_equal(out[:, 2], down.T)


@pytest.mark.parametrize("reuse", [True, False])
@pytest.mark.parametrize("N,C,k,B", [(12, 5, 3, 1), (40, 20, 8, 1), (16, 6, 2, 4), (60, 30, 4, 32), (8, 4, 2, 1)])
def test_slot_planner_matches_oracle_slot_cache(lib, N, C, k, B, reuse):
    rng = np.random.default_rng(N * 1000 + C * 10 + B + int(reuse))
    host = binding.Slots(N, C, reuse)
    orc = ao.SlotCache(N, C, cache_reuse=reuse)
    for step in range(150):
        host.begin_step(); orc.begin_step()
        cands = []
        for b in range(B):
            n = int(rng.integers(k, C + 1))
            cands.append([int(e) for e in rng.choice(N, size=n, replace=False)])
        U, ocp = orc.prefetch(cands)
        hcp = host.prefetch(cands)
        assert hcp == ocp
        if step % 3 == 0:       # stall-free style step: touch some residents
            R = orc.resident()
            used = [int(e) for e in rng.choice(R, size=min(k, len(R)), replace=False)]
            for e in sorted(used):
                orc.touch(e)
            host.touch(used)
        else:                   # exact style step
            K = [[int(e) for e in rng.choice(N, size=k, replace=False)] for _ in range(B)]
            missing, waves = orc.demand(K)
            hd = host.demand(K)
            flat = [(e, s, w + 1) for w, wv in enumerate(waves) for (e, s) in wv]
            assert hd == flat
        es, st, clk = host.get()
        assert list(es) == orc.expert_slot and list(st) == orc.slot_stamp and clk == orc.clock


def test_slot_planner_set_rejects_inconsistent_tables(lib):
    s = binding.Slots(4, 2)
    assert s.set([0, 0, -1, -1], [0, 0], 1) == binding.APEX_EINVAL      # two experts in slot 0
    assert s.set([0, 5, -1, -1], [0, 0], 1) == binding.APEX_EINVAL      # slot out of range
    assert s.set([1, -1, 0, -1], [3, 4], 7) == 0
    es, st, clk = s.get()
    assert list(es) == [1, -1, 0, -1] and list(st) == [3, 4] and clk == 7
