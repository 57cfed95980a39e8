"""Seeded synthetic inputs with the shapes of the paper's models.

This module only draws random tensors (and loads the frozen confidence-model parameters
that were fitted offline).  It contains none of the method's arithmetic: no router
product, no softmax, no ranking, no expert FFN.  Both the CPU oracle's tests and the
CUDA path's tests / benchmark take their inputs from here, so that the two sides see
identical bytes without sharing any code of the method.

Recipe (one base seed, one sub-stream per (config, layer, tensor kind)):

* router            W_r ~ N(0, 1/d) fp32; optional bias b_r = 0.5*ln f_e, f_e a Zipf(s=1.1)
                    frequency over a seeded permutation of the experts (skewed popularity)
* prefetch router   W_p = W_r + N(0, sigma_p^2/d), b_p = b_r  (it mirrors the router)
* hidden states     h ~ N(0,1); h' = h + N(0, 0.25); both rounded to bf16-representable
                    values but stored widened in fp32
* expert weights    bf16, N(0, 0.02^2), generated directly in the library's store layout
                    [I][3][d]: for intermediate index i the rows gate_i, up_i, downT_i
                    (downT is W_down transposed)
* confidence model  w[N], theta[N-k+1]: frozen values fitted offline on calibration tokens
                    of this same generator (files under ``data/``), else a fixed hand-set
                    model
"""
from __future__ import annotations

import dataclasses
import os
from typing import Optional, Tuple

import numpy as np

BASE_SEED = 11688

_KIND = {"router": 1, "prefetch_noise": 2, "hidden": 3, "hidden_noise": 4, "experts": 5,
         "shared": 6, "zipf_perm": 7, "calib_hidden": 8, "calib_noise": 9, "attn": 10}


@dataclasses.dataclass(frozen=True)
class Config:
    cfg_id: int
    name: str
    L: int          # layers
    d: int          # hidden size
    N: int          # experts per layer
    k: int          # routed experts per token
    I: int          # expert intermediate size
    C: int          # HBM cache slots per layer
    T: int          # decode steps
    batches: Tuple[int, ...] = (1,)
    I_shared: int = 0
    sigma_p: float = 0.3      # prefetch-router noise std, in units of 1/sqrt(d)
    hidden_noise: float = 0.5  # std of h' - h per element (what attention adds that the prefetch router cannot see)
    zipf_s: float = 0.0       # >0: skewed expert popularity through a router bias
    modes: Tuple[str, ...] = ("exact", "stall_free")

    @property
    def expert_bytes(self) -> int:
        return 3 * self.d * self.I * 2

    @property
    def shared_bytes(self) -> int:
        return 3 * self.d * self.I_shared * 2

    def scaled(self, **kw) -> "Config":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    0: Config(0, "tiny-granite1b-layer", L=1, d=1024, N=32, k=8, I=512, C=16, T=128,
              modes=("exact",)),
    1: Config(1, "granite-3b-a800m-shape", L=32, d=1536, N=40, k=8, I=512, C=20, T=1024),
    2: Config(2, "olmoe-shape", L=16, d=2048, N=64, k=8, I=1024, C=24, T=2048, zipf_s=1.1),
    3: Config(3, "mixtral-8x7b-shape", L=32, d=4096, N=8, k=2, I=14336, C=4, T=512,
              sigma_p=0.5),
    4: Config(4, "qwen1.5-moe-shape", L=24, d=2048, N=60, k=4, I=1408, C=30, T=64,
              batches=(1, 8, 32, 128, 256), I_shared=5632, modes=("exact",)),
}


def _rng(cfg: Config, layer: int, kind: str) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([BASE_SEED, cfg.cfg_id, layer, _KIND[kind]]))


def round_to_bf16_values(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16-representable value (ties to even), keep fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    bias = 0x7FFF + ((u >> 16) & 1)
    u = ((u + bias) & 0xFFFF0000).astype(np.uint32)
    return u.view(np.float32).reshape(x.shape)


def router_weights(cfg: Config, layer: int):
    """Returns (W_r [N][d], b_r [N], W_p [N][d], b_p [N]) as fp32 arrays."""
    d, N = cfg.d, cfg.N
    W_r = (_rng(cfg, layer, "router").standard_normal((N, d)) / np.sqrt(d)).astype(np.float32)
    noise = _rng(cfg, layer, "prefetch_noise").standard_normal((N, d)) * (cfg.sigma_p / np.sqrt(d))
    W_p = (W_r.astype(np.float64) + noise).astype(np.float32)
    if cfg.zipf_s > 0:
        perm = _rng(cfg, layer, "zipf_perm").permutation(N)          # perm[e] = popularity rank - 1
        f = (perm + 1.0) ** (-cfg.zipf_s)
        f /= f.sum()
        b_r = (0.5 * np.log(f)).astype(np.float32)
    else:
        b_r = np.zeros(N, dtype=np.float32)
    return W_r, b_r, W_p, b_r.copy()


def hidden_states(cfg: Config, layer: int, T: int, B: int = 1, calib: bool = False):
    """Returns (h [T][B][d], h' [T][B][d]) fp32 holding bf16-representable values."""
    a, b = ("calib_hidden", "calib_noise") if calib else ("hidden", "hidden_noise")
    h = _rng(cfg, layer, a).standard_normal((T, B, cfg.d)).astype(np.float32)
    hp = h + np.float32(cfg.hidden_noise) * _rng(cfg, layer, b).standard_normal((T, B, cfg.d)).astype(np.float32)
    return round_to_bf16_values(h), round_to_bf16_values(hp)


def expert_store(cfg: Config, layer: int, device="cpu", pin: bool = False, out=None):
    """bf16 tensor [N][I][3][d] in the library's store layout: per intermediate index i the rows
    gate_i, up_i, downT_i.

    The conceptual down projection is W_down[j][i] = downT[i][j] = store[e][i][2][j].  Drawn with torch's
    seeded generator on ``device`` (CPU and CUDA streams differ; within one run everybody
    reads the same bytes).
    """
    import torch
    shape = (cfg.N, cfg.I, 3, cfg.d)
    g = torch.Generator(device=device)
    g.manual_seed((BASE_SEED * 1000003 + cfg.cfg_id * 10007 + layer * 101 + _KIND["experts"]) & 0x7FFFFFFF)
    if out is None:
        out = torch.empty(shape, dtype=torch.bfloat16, device="cpu", pin_memory=pin) \
            if str(device) == "cpu" else torch.empty(shape, dtype=torch.bfloat16, device=device)
    # draw expert by expert to bound the fp32 temporary
    for e in range(cfg.N):
        t = torch.randn((cfg.I, 3, cfg.d), generator=g, device=device, dtype=torch.float32)
        out[e].copy_((t * 0.02).to(torch.bfloat16))
    return out


def shared_expert(cfg: Config, layer: int, device="cpu"):
    """bf16 tensor [I_shared][3][d] (rows gate_i, up_i, downT_i) or None when the config has none."""
    import torch
    if cfg.I_shared == 0:
        return None
    g = torch.Generator(device=device)
    g.manual_seed((BASE_SEED * 1000003 + cfg.cfg_id * 10007 + layer * 101 + _KIND["shared"]) & 0x7FFFFFFF)
    t = torch.randn((cfg.I_shared, 3, cfg.d), generator=g, device=device, dtype=torch.float32)
    return (t * 0.02).to(torch.bfloat16)


def handset_cdf_params(cfg: Config):
    """A fixed, monotone confidence model used when no fitted file exists.

    x is the prefetch distribution sorted in descending order.  Probability mass just below
    the top-k boundary raises the latent score (less confident, larger budget); mass inside
    the top-k lowers it.
    """
    N, k = cfg.N, cfg.k
    w = np.zeros(N, dtype=np.float32)
    w[:k] = -2.0
    w[k:min(N, 2 * k)] = 6.0
    theta = (-1.0 + 0.6 * np.arange(N - k + 1)).astype(np.float32)
    return w, theta


_DATA_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "data")


def cdf_params(cfg: Config, layer: int, allow_handset: bool = True):
    """(w [N], theta [N-k+1]) fp32: the frozen confidence model of this config and layer."""
    path = os.path.join(_DATA_DIR, f"cdf_cfg{cfg.cfg_id}.npz")
    if os.path.exists(path):
        z = np.load(path)
        if z["w"].shape == (cfg.L, cfg.N) and layer < cfg.L:
            return z["w"][layer].astype(np.float32), z["theta"][layer].astype(np.float32)
    if not allow_handset:
        raise FileNotFoundError(path)
    return handset_cdf_params(cfg)


def split_store(w):
    """Store layout [..., I, 3, d] -> the usual (W_gate [I][d], W_up [I][d], W_down [d][I]) views."""
    return w[..., 0, :], w[..., 1, :], np.swapaxes(w[..., 2, :], -1, -2)


def quantize_store_fp8(w):
    """bf16/fp32 store [..., I, 3, d] -> uint8 [..., I, 3*d + 16] in the library's e4m3 row layout.

    Per row (one of gate_i, up_i, downT_i) the scale is max|row| / 448 (448 = largest e4m3 value; 1 for an all-zero
    row), the codes are the row divided by its scale, rounded to e4m3 by torch's cast.  A row block is
    3*d code bytes, then the three fp32 scales, then 4 zero bytes.
    """
    import torch
    wf = w.to(torch.float32)
    d = wf.shape[-1]
    amax = wf.abs().amax(dim=-1, keepdim=True)
    scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax))
    codes = (wf / scale).to(torch.float8_e4m3fn).view(torch.uint8)             # [..., I, 3, d]
    lead = codes.shape[:-2]
    out = torch.zeros(lead + (3 * d + 16,), dtype=torch.uint8, device=w.device)
    out[..., :3 * d] = codes.reshape(lead + (3 * d,))
    sc = torch.zeros(lead + (4,), dtype=torch.float32, device=w.device)
    sc[..., :3] = scale.squeeze(-1)
    out[..., 3 * d:] = sc.view(torch.uint8).reshape(lead + (16,))
    return out


def dequantize_store_fp8(q, d: int) -> np.ndarray:
    """uint8 [..., I, 3*d + 16] -> fp64 numpy [..., I, 3, d]: weight = scale * code, multiplied in fp64 (the
    product of an e4m3 value and an fp32 scale is exact there)."""
    import torch
    q = q.detach().cpu()
    lead = q.shape[:-1]
    codes = q[..., :3 * d].contiguous().view(torch.float8_e4m3fn).to(torch.float32).reshape(lead + (3, d)).numpy()
    sc = q[..., 3 * d:].contiguous().view(torch.float32)[..., :3].numpy()
    return codes.astype(np.float64) * sc[..., None].astype(np.float64)


def expert_store_fp8(cfg: Config, layer: int, device="cpu"):
    """uint8 tensor [N][I][3*d+16]: the seeded bf16 store of ``expert_store`` quantised row by row."""
    import torch
    out = torch.empty((cfg.N, cfg.I, 3 * cfg.d + 16), dtype=torch.uint8, device=device)
    g = torch.Generator(device=device)
    g.manual_seed((BASE_SEED * 1000003 + cfg.cfg_id * 10007 + layer * 101 + _KIND["experts"]) & 0x7FFFFFFF)
    for e in range(cfg.N):
        t = torch.randn((cfg.I, 3, cfg.d), generator=g, device=device, dtype=torch.float32)
        out[e].copy_(quantize_store_fp8((t * 0.02).to(torch.bfloat16)))
    return out


_E2M1 = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)


def fp4_row_bytes(d: int) -> int:
    """Bytes of one intermediate index in the block-scaled e2m1 layout: codes, block scales, padding to 16."""
    return (3 * (d // 2) + 3 * (d // 32) + 15) & ~15


def quantize_store_fp4(w):
    """bf16/fp32 store [..., I, 3, d] -> uint8 [..., I, fp4_row_bytes(d)] in the library's block-scaled e2m1 layout.

    Per block of 32 consecutive elements of a vector the scale is the power of two 2^e with e the smallest integer
    for which max|block| / 2^e <= 6 (6 = largest e2m1 value), stored as the byte e + 127 (0 for an all-zero block:
    scale 0).  Codes: sign bit and the index of the nearest of (0, .5, 1, 1.5, 2, 3, 4, 6); two per byte, the even
    element in the low nibble.  Row: gate | up | downT codes (d/2 bytes each), then their scale bytes (d/32 each).
    """
    import torch
    wf = w.to(torch.float32)
    d = wf.shape[-1]
    lead = wf.shape[:-2]
    blk = wf.reshape(lead + (3, d // 32, 32))
    amax = blk.abs().amax(dim=-1)
    e = torch.ceil(torch.log2(torch.clamp(amax, min=1e-38) / 6.0))
    e = torch.clamp(e, -126, 127)
    sbyte = torch.where(amax > 0, e + 127, torch.zeros_like(e)).to(torch.uint8)                  # [..., 3, d/32]
    scale = torch.where(amax > 0, torch.exp2(e), torch.ones_like(e))
    x = blk / scale[..., None]
    mids = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=torch.float32, device=wf.device)
    code = torch.bucketize(x.abs(), mids).to(torch.uint8) | ((x < 0).to(torch.uint8) << 3)         # [..., 3, d/32, 32]
    code = code.reshape(lead + (3, d // 2, 2))
    packed = code[..., 0] | (code[..., 1] << 4)                                                     # [..., 3, d/2]
    out = torch.zeros(lead + (fp4_row_bytes(d),), dtype=torch.uint8, device=wf.device)
    out[..., :3 * (d // 2)] = packed.reshape(lead + (3 * (d // 2),))
    out[..., 3 * (d // 2):3 * (d // 2) + 3 * (d // 32)] = sbyte.reshape(lead + (3 * (d // 32),))
    return out


def dequantize_store_fp4(q, d: int) -> np.ndarray:
    """uint8 [..., I, fp4_row_bytes(d)] -> fp64 numpy [..., I, 3, d]: weight = 2^(scale byte - 127) * code value
    (scale byte 0: the block is zero)."""
    q = q.detach().cpu().numpy()
    lead = q.shape[:-1]
    packed = q[..., :3 * (d // 2)].reshape(lead + (3, d // 2))
    codes = np.stack([packed & 0xF, packed >> 4], axis=-1).reshape(lead + (3, d))
    table = np.array(_E2M1 + tuple(-v for v in _E2M1), dtype=np.float64)
    vals = table[codes]
    sb = q[..., 3 * (d // 2):3 * (d // 2) + 3 * (d // 32)].reshape(lead + (3, d // 32)).astype(np.int64)
    scale = np.where(sb > 0, np.ldexp(1.0, sb - 127), 0.0)
    return vals * np.repeat(scale, 32, axis=-1)


def expert_store_fp4(cfg: Config, layer: int, device="cpu"):
    """uint8 tensor [N][I][fp4_row_bytes(d)]: the seeded bf16 store of ``expert_store`` quantised block by block."""
    import torch
    out = torch.empty((cfg.N, cfg.I, fp4_row_bytes(cfg.d)), dtype=torch.uint8, device=device)
    g = torch.Generator(device=device)
    g.manual_seed((BASE_SEED * 1000003 + cfg.cfg_id * 10007 + layer * 101 + _KIND["experts"]) & 0x7FFFFFFF)
    for e in range(cfg.N):
        t = torch.randn((cfg.I, 3, cfg.d), generator=g, device=device, dtype=torch.float32)
        out[e].copy_(quantize_store_fp4((t * 0.02).to(torch.bfloat16)))
    return out


def bf16_to_f32_numpy(t) -> np.ndarray:
    """Lossless widening of a torch bf16 tensor to a numpy fp32 array (test helper)."""
    import torch
    return t.detach().to("cpu").to(torch.float32).numpy()


def tiny_config(d=256, N=8, k=2, I=64, C=4, L=1, T=8, I_shared=0, sigma_p=0.3, zipf_s=0.0,
                cfg_id=100, batches=(1,)) -> Config:
    """Small shapes for brute-force tests."""
    return Config(cfg_id, "tiny", L=L, d=d, N=N, k=k, I=I, C=C, T=T, batches=batches,
                  I_shared=I_shared, sigma_p=sigma_p, zipf_s=zipf_s)
