"""Seeded synthetic inputs shaped like the paper's workload.

This module holds NO arithmetic of the method (no quantisation, no sorting, no
attention): it only draws tensors.  It is the one module that the tests hand
to both the CUDA library and the CPU oracle.

Value law (Sec. II-C, Sec. IV of the paper: key outliers sit in a few channels
per head, consistent across tokens and sequences): every element ~ N(0, 1);
in each KV head ``n_outliers`` distinct seeded channels of K are multiplied by
a per-channel scale, fixed (x20) in the small single-head case and
~LogNormal(mu=2.5, sigma=0.5) in the model-shaped cases.  Shapes follow
Llama-2-7B (32 heads x 128) and a Llama-3-8B-like GQA layer (32 query heads,
8 KV heads).  The paper's real data (Llama-2-7B keys on wikitext-2) is not
available offline; these tensors stand in for it.

Seeds: 20137 + 1000 * config + {0: K, 1: V, 2: q, 3: outlier channels,
4: outlier scales, 5: calibration tokens}.
"""
from dataclasses import dataclass, field
from typing import Optional, Tuple

import numpy as np
import torch

BASE_SEED = 20137
K_STREAM, V_STREAM, Q_STREAM, CHAN_STREAM, SCALE_STREAM, CALIB_STREAM = range(6)


@dataclass(frozen=True)
class Workload:
    """One named configuration (index = position in the benchmark's config list, 1-based)."""
    config: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq: int                      # cached tokens attended over
    dtype: str                    # "f32" | "bf16"
    block: int
    mant_bits: int
    n_outliers: int
    fixed_outliers: Optional[Tuple[int, ...]] = None   # config 1: fixed channels, x20
    fixed_scale: float = 20.0
    calib_tokens: int = 0
    note: str = field(default="", compare=False)


CONFIGS = {
    1: Workload(1, 1, 1, 1, 128, 256, "f32", 16, 4, 4, fixed_outliers=(3, 37, 74, 120),
                calib_tokens=256, note="single head, 4 fixed outlier channels x20"),
    2: Workload(2, 1, 32, 32, 128, 4096, "bf16", 32, 4, 6, calib_tokens=4096,
                note="Llama-2-7B-shaped layer, batch 1"),
    3: Workload(3, 16, 32, 32, 128, 8192, "bf16", 32, 4, 6, calib_tokens=4096,
                note="Llama-2-7B-shaped layer, batch 16, append 1 + decode"),
    4: Workload(4, 8, 32, 8, 128, 32768, "bf16", 32, 4, 8, calib_tokens=4096,
                note="Llama-3-8B-shaped GQA layer, batch 8"),
    5: Workload(5, 1, 8, 8, 128, 65536, "bf16", 32, 4, 6, calib_tokens=1 << 20,
                note="prefill/append and calibration sweep"),
}


def seed_for(config: int, stream: int) -> int:
    return BASE_SEED + 1000 * config + stream


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def outlier_channels(w: Workload, device="cpu"):
    """-> (channels int64 [H_kv, n_out], scales f32 [H_kv, n_out]); drawn on the host so that
    the same channels are used whatever device the big tensors are drawn on."""
    H, n_out, d = w.n_kv_heads, w.n_outliers, w.head_dim
    if w.fixed_outliers is not None:
        ch = torch.tensor([list(w.fixed_outliers)] * H, dtype=torch.int64)
        sc = torch.full((H, n_out), w.fixed_scale, dtype=torch.float32)
    else:
        gc = _gen("cpu", seed_for(w.config, CHAN_STREAM))
        ch = torch.stack([torch.randperm(d, generator=gc)[:n_out] for _ in range(H)])
        gs = _gen("cpu", seed_for(w.config, SCALE_STREAM))
        sc = torch.exp(2.5 + 0.5 * torch.randn(H, n_out, generator=gs, dtype=torch.float32))
    return ch.to(device), sc.to(device)


def channel_scale(w: Workload, device="cpu") -> torch.Tensor:
    """Per-(head, channel) multiplier [H_kv, d] f32: 1 everywhere except the outlier channels."""
    ch, sc = outlier_channels(w, device)
    m = torch.ones(w.n_kv_heads, w.head_dim, dtype=torch.float32, device=device)
    m.scatter_(1, ch, sc)
    return m


def _normal_scaled(shape, seed, device, dtype, mult=None, chunk_tokens=1 << 16):
    """N(0,1) of ``shape`` = [..., tokens, H, d], optionally times mult[H, d], rounded once to
    ``dtype``.  Drawn in token chunks so a multi-GB tensor needs little fp32 scratch."""
    g = _gen(device, seed)
    out = torch.empty(shape, dtype=dtype, device=device)
    flat = out.view(-1, shape[-2], shape[-1])
    for t0 in range(0, flat.shape[0], chunk_tokens):
        t1 = min(flat.shape[0], t0 + chunk_tokens)
        x = torch.randn(t1 - t0, shape[-2], shape[-1], generator=g, device=device, dtype=torch.float32)
        if mult is not None:
            x *= mult
        flat[t0:t1] = x.to(dtype)
    return out


def make_kv(w: Workload, n_tokens: Optional[int] = None, device="cpu", outliers_in_v: bool = False,
            batch: Optional[int] = None):
    """K, V of shape [B, n_tokens, H_kv, d] (the layout the append call takes)."""
    T = w.seq if n_tokens is None else n_tokens
    B = w.batch if batch is None else batch
    mult = channel_scale(w, device)
    shape = (B, T, w.n_kv_heads, w.head_dim)
    dt = torch_dtype(w.dtype)
    k = _normal_scaled(shape, seed_for(w.config, K_STREAM), device, dt, mult)
    v = _normal_scaled(shape, seed_for(w.config, V_STREAM), device, dt, mult if outliers_in_v else None)
    return k, v


def make_q(w: Workload, device="cpu", batch: Optional[int] = None):
    """q of shape [B, H_q, d]."""
    B = w.batch if batch is None else batch
    g = _gen(device, seed_for(w.config, Q_STREAM))
    q = torch.randn(B, w.n_q_heads, w.head_dim, generator=g, device=device, dtype=torch.float32)
    return q.to(torch_dtype(w.dtype))


def make_calibration(w: Workload, n_tokens: Optional[int] = None, device="cpu"):
    """Calibration keys [T, H_kv, d] with the same outlier channels, their own seed."""
    T = w.calib_tokens if n_tokens is None else n_tokens
    mult = channel_scale(w, device)
    return _normal_scaled((T, w.n_kv_heads, w.head_dim), seed_for(w.config, CALIB_STREAM), device,
                          torch_dtype(w.dtype), mult)


def to_oracle(x: torch.Tensor) -> np.ndarray:
    """Host copy in the form the oracle takes: f32 as float32, bf16 as uint16 bit patterns."""
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16)
    return x.numpy()
