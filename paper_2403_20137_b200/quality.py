"""Quality report of the BFP cache with and without channel sorting (Sec. II-C first paragraph: a block that
holds an outlier rounds its small elements towards zero; Table I: sorting lowers the damage at the same bits;
Sec. III last paragraph: the same idea on the value side).

Everything that is measured runs through the CUDA library: the cache is written by ``kvbfp_append``, read back by
``kvbfp_dequant`` and attended over by ``kvbfp_decode_attn``.  Only the yardstick -- attention over the
UNQUANTISED keys and values -- is plain fp32 torch on the same device; it is not part of the path.

All figures are averaged over every KV head (and query head) of the configuration:

* ``key_mse`` / ``value_mse``: mean squared error of the dequantised cache against what was appended;
* ``score_rms_err``: root mean square error of the pre-softmax scores q.k (unscaled);
* ``attn_out_rel_err``: per (batch, query head) row, max_c |o - o_ref| / max_c |o_ref| against unquantised
  attention, mean and maximum over the rows.
"""
import dataclasses
import math

import torch

from . import binding as B
from . import workloads as W


def _rows_rel_err(o, ref):
    num = (o - ref).abs().amax(dim=-1)
    den = ref.abs().amax(dim=-1).clamp_min(1e-30)
    r = num / den
    return float(r.mean()), float(r.max())


def _plain_attention(q, k, v, scale):
    """q [B, Hq, d], k/v [B, T, Hkv, d] (any float dtype) -> fp32 [B, Hq, d], scores [B, Hq, T] (unscaled)."""
    Bn, T, Hkv, d = k.shape
    G = q.shape[1] // Hkv
    kf = k.float().permute(0, 2, 1, 3)                        # [B, Hkv, T, d]
    vf = v.float().permute(0, 2, 1, 3)
    qf = q.float().view(Bn, Hkv, G, d)
    s = torch.einsum("bhgd,bhtd->bhgt", qf, kf)
    p = torch.softmax(s * scale, dim=-1)
    o = torch.einsum("bhgt,bhtd->bhgd", p, vf)
    return o.reshape(Bn, Hkv * G, d), s.reshape(Bn, Hkv * G, T)


def _one_side(w, k, v, q, perm_k, perm_v, inv_perm_v, ref_o, ref_s, scale, per_head=False):
    Bn, T, Hkv, d = k.shape
    dev = k.device
    cache = B.Cache(Bn, Hkv, d, (T + 15) // 16 * 16, w.block, w.mant_bits, device=dev)
    z = torch.zeros(Bn, dtype=torch.int32, device=dev)
    B.append(cache, k, v, z, perm_k=perm_k, perm_v=perm_v)
    kd = B.dequant_all(cache, "k", T, perm=perm_k)
    vd = B.dequant_all(cache, "v", T, perm=perm_v)
    lens = torch.full((Bn,), T, dtype=torch.int32, device=dev)
    o = B.decode_attn(cache, q, lens, perm_k=perm_k, inv_perm_v=inv_perm_v, softmax_scale=scale)
    G = q.shape[1] // Hkv
    s = torch.einsum("bhgd,bthd->bhgt", q.float().view(Bn, Hkv, G, d), kd).reshape(Bn, Hkv * G, T)
    mean_e, max_e = _rows_rel_err(o, ref_o)
    extra = {}
    if per_head:
        extra = {"key_mse_per_head": [float(x) for x in ((kd - k.float()) ** 2).mean(dim=(0, 1, 3))],
                 "value_mse_per_head": [float(x) for x in ((vd - v.float()) ** 2).mean(dim=(0, 1, 3))],
                 "attn_out": o}
    return {**extra, "key_mse": float(((kd - k.float()) ** 2).mean()), "value_mse": float(((vd - v.float()) ** 2).mean()),
            "score_rms_err": float(((s - ref_s) ** 2).mean().sqrt()),
            "attn_out_rel_err_mean": mean_e, "attn_out_rel_err_max": max_e}


def quality_report(w: W.Workload, device="cuda", n_tokens=2048, batch=1, outliers_in_v=False, sort_v=False,
                   per_head=False, draw_on=None):
    """Cache quality of configuration ``w`` on ``batch`` sequences of ``n_tokens`` tokens, all heads: unsorted
    BFP against K-sorted BFP (and V-sorted, with ``sort_v``), same bits.  The permutations come from
    ``kvbfp_calibrate`` over the configuration's calibration tokens (keys) and over the appended values
    themselves (values: the paper postpones the value side and names no calibration set for it).  ``per_head``
    adds the per-head errors and the attention output tensors (for tests); ``draw_on`` names the device whose
    generator draws the inputs (the host's and the GPU's streams differ for one seed), default ``device``."""
    w1 = dataclasses.replace(w, batch=batch)
    src = device if draw_on is None else draw_on
    k, v = (x.to(device) for x in W.make_kv(w1, n_tokens=n_tokens, device=src, outliers_in_v=outliers_in_v))
    q = W.make_q(w1, device=src).to(device)
    Hkv, d = w.n_kv_heads, w.head_dim
    calib = W.make_calibration(w, n_tokens=min(w.calib_tokens, 4096), device=src).to(device)
    _, perm_k, _ = B.calibrate(calib, Hkv, d)
    perm_v = inv_perm_v = None
    if sort_v:
        _, perm_v, inv_perm_v = B.calibrate(v.reshape(-1, Hkv, d), Hkv, d)
    scale = 1.0 / math.sqrt(d)
    ref_o, ref_s = _plain_attention(q, k, v, scale)
    rep = {"tokens": n_tokens, "sequences": batch, "kv_heads": Hkv, "q_heads": w.n_q_heads,
           "block": w.block, "mant_bits": w.mant_bits, "bits_per_element": w.mant_bits + 8.0 / w.block,
           "outliers_in_v": outliers_in_v,
           "unsorted": _one_side(w, k, v, q, None, None, None, ref_o, ref_s, scale, per_head),
           "ksort": _one_side(w, k, v, q, perm_k, None, None, ref_o, ref_s, scale, per_head)}
    if per_head:
        rep["unquantised_out"] = ref_o
    if sort_v:
        rep["ksort_vsort"] = _one_side(w, k, v, q, perm_k, perm_v, inv_perm_v, ref_o, ref_s, scale, per_head)
    return rep
