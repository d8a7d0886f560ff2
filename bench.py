"""Benchmark of the BFP KV-cache decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 3]

One "step" is one generated token for every sequence of the batch through the cache path:
kvbfp_append of the new token's K and V (1 token per sequence) followed by kvbfp_decode_attn over
the whole cached sequence.  The permutation (kvbfp_calibrate) is found once before the loop: by the
method's own account it is fixed before inference starts.  The workload is the Llama-2-7B-shaped
layer with batch 16 and 8192 cached tokens, block 32, 4-bit mantissas, synthetic outlier-structured
bf16 keys.  With N > 1 (torchrun) every rank owns its own batch of sequences and there is no
data-path collective (weak scaling); time is the max over ranks.

Prints ONE JSON line on rank 0.
"""
import argparse
import dataclasses
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2403_20137_b200 import workloads as W  # noqa: E402

METRIC = "decode_attn_tokens_per_s"
UNIT = "tokens/s"

# DRAM traffic of the dominant kernel from one ncu capture per kernel (batch 4 of the same shape; the summaries of
# those captures are kept under profiles/):
# dram__bytes_read.sum + dram__bytes_write.sum per (batch, kv head, token) unit on a smaller case of the
# same kernel, scaled by the units of a launch.  Valid only while the kernel sources still hash to the
# value recorded with the capture; otherwise the bench reports null.
TRAFFIC = {"decode_mma4": {"bytes_per_unit": 138.2494, "block": 32, "mant_bits": 4, "sources_sha256": "3006fc386180fab06b257266496bbd0efb400e9c00028bf7c6fd405c7e93f5b1"},
           "decode_mma8": {"bytes_per_unit": 265.9599, "block": 32, "mant_bits": 8, "sources_sha256": "6ed4258b1fccf49c444f7130c499314796c7f5a30bf680a283449208da4f8c57"},
           "decode_mma6": {"bytes_per_unit": 201.705, "block": 32, "mant_bits": 6, "sources_sha256": "67627b858a3acb111ed91753e2373c139cfb0c3d831bb95f444c7884b64c04dc"}}
KERNEL_SOURCES = {"decode_mma4": ["paper_2403_20137_b200/csrc/decode_mma4.cu", "paper_2403_20137_b200/csrc/ptx.cuh"],
                  "decode_mma8": ["paper_2403_20137_b200/csrc/decode_mma8.cu", "paper_2403_20137_b200/csrc/ptx.cuh"],
                  "decode_mma6": ["paper_2403_20137_b200/csrc/decode_mma6.cu", "paper_2403_20137_b200/csrc/ptx.cuh"]}


def sources_hash(kernel):
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES.get(kernel, []):
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def traffic_per_launch(kernel, w):
    """DRAM bytes of one launch, scaled from the capture by the units processed; None when there is no capture for
    this kernel and format or the kernel has changed since."""
    t = TRAFFIC.get(kernel)
    if not t or not t["bytes_per_unit"] or (w.block, w.mant_bits) != (t["block"], t["mant_bits"]) or \
            t["sources_sha256"] != sources_hash(kernel):
        return None
    return t["bytes_per_unit"] * decode_units(w)


def workload_name(w):
    return (f"config{w.config}: B{w.batch} Hq{w.n_q_heads} Hkv{w.n_kv_heads} d{w.head_dim} S{w.seq} {w.dtype} "
            f"BFP block{w.block} mant{w.mant_bits}; append 1 token/seq + decode attention")


def config_of(w):
    """The `config` object of both arms: the workload, and how the L2 is kept out of the timing."""
    return {"workload": workload_name(w),
            "l2": f"inputs larger than L2: {decode_bytes(w) / 1e6:.0f} MB of cache read per step vs 126 MB L2"}


def decode_units(w):
    return w.batch * w.n_kv_heads * w.seq


def decode_bytes(w):
    """Algorithmic bytes of one decode launch: packed K and V rows of every cached token, once."""
    row = w.head_dim * w.mant_bits // 8 + w.head_dim // w.block
    return 2 * row * decode_units(w)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy bandwidth)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier copy measurement on this pool)"


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_throughput(per_rank_units, world, ms_per_step_max):
    """Units all ranks processed per second, timed by the slowest rank."""
    return world * per_rank_units / (ms_per_step_max * 1e-3)


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for n, v in zip(names, r[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


class OracleStep:
    """The CPU oracle, as it stands, on `n_units` (batch, kv head) units of one step of the workload:
    append of the new token and decode attention over the full sequence.  Units are independent and
    are spread over the host cores with threads (the C oracle runs outside the GIL)."""

    def __init__(self, w, n_units):
        import numpy as np

        import oracle as O
        O.lib()
        self.O, self.np, self.w = O, np, w
        self.cores = max(1, min(os.cpu_count() or 1, n_units))
        S, d = w.seq, w.head_dim
        self.G = w.n_q_heads // w.n_kv_heads
        # one kv head at a time: [1, S, 1, d] tensors drawn by the same seeded generators as the GPU arm
        one = W.Workload(w.config, 1, self.G, 1, d, S, w.dtype, w.block, w.mant_bits, w.n_outliers)
        k, v = W.make_kv(one, n_tokens=S)
        self.kn, self.vn, self.qn = W.to_oracle(k), W.to_oracle(v), W.to_oracle(W.make_q(one))
        _, self.perm, _ = O.calibrate(self.kn.reshape(S, 1, d), w.dtype, 1, d)
        self.caches = []
        for _ in range(n_units):
            c = O.Cache(1, 1, d, S, w.block, w.mant_bits)
            O.append(c, self.kn[:, :S - 1], self.vn[:, :S - 1], w.dtype, np.zeros(1, np.int32), perm_k=self.perm)
            self.caches.append(c)        # prefill is set-up, not timed

    def _unit(self, c):
        O, np, S, w = self.O, self.np, self.w.seq, self.w
        O.append(c, self.kn[:, S - 1:], self.vn[:, S - 1:], w.dtype, np.array([S - 1], np.int32), perm_k=self.perm)
        return O.decode_attn(c, self.qn, w.dtype, self.G, [S], perm_k=self.perm)

    def run(self):
        from concurrent.futures import ThreadPoolExecutor
        t0 = time.perf_counter()
        with ThreadPoolExecutor(max_workers=self.cores) as ex:
            list(ex.map(self._unit, self.caches))
        return time.perf_counter() - t0


def run_reference(args, w, rank):
    """The reference arm is the CPU oracle, timed as it stands on the host cores (rank 0 only).  Each
    step is a bounded sample of the workload, sized so that the whole run takes a couple of minutes."""
    if rank != 0:
        return
    n_units = w.batch * w.n_kv_heads
    probe = OracleStep(w, 1)
    t_unit = min(probe.run() for _ in range(2))
    ncores = os.cpu_count() or 1
    budget_s = 100.0
    sample = int(budget_s * ncores / (t_unit * max(1, args.steps + args.warmup)))
    sample = max(1, min(sample, n_units))
    if args.ref_units:
        sample = max(1, min(args.ref_units, n_units))
    st = OracleStep(w, sample)
    for _ in range(args.warmup):
        st.run()
    times = [st.run() for _ in range(args.steps)]
    t_step_full = statistics.mean(times) * n_units / sample        # scaled to all (batch, head) units
    value = w.batch / t_step_full
    desc = (f"{sample} of {n_units} (batch, kv head) units of one step (append 1 token + decode over {w.seq} "
            f"tokens), time scaled to all units")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t_step_full, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": st.cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def sweep_config5(B, dev):
    """Prefill/append and calibration sweep: 8 KV heads x 128, 65536 new bf16 tokens with the outlier law,
    calibration (max-abs + argsort) over 2^20 tokens, append throughput and key MSE with/without K-sort for
    blocks 16/32/64 x mantissas 4/6/8."""
    w = W.CONFIGS[5]
    H, d, T = w.n_kv_heads, w.head_dim, w.seq
    out = {}
    calib = W.make_calibration(w, device=dev)                       # [2^20, 8, 128] bf16 = 2 GiB
    _, perm, _ = B.calibrate(calib, H, d)
    ms = timed(lambda: B.calibrate(calib, H, d), reps=3)
    out["calibrate"] = {"tokens": int(calib.shape[0]), "ms": ms, "GB/s": calib.numel() * 2 / ms / 1e6}
    # the paper's own front end: Euclidean norm of the rows of W_k (given transposed, [d_in, H*d]), rows folded by the
    # permutation (Algorithm 1 steps 1, 3-4)
    wk_t = calib[:4096]                                             # stands in for W_k^T: [4096, 8, 128]
    _, perm_l2, _ = B.calibrate(wk_t, H, d, stat=B.STAT_L2)
    ms = timed(lambda: B.calibrate(wk_t, H, d, stat=B.STAT_L2), reps=5)
    out["calibrate_l2"] = {"rows": 4096, "ms": ms, "GB/s": wk_t.numel() * 2 / ms / 1e6}
    wk = torch.randn(H * d, 4096, dtype=torch.bfloat16, device=dev, generator=torch.Generator(device=dev).manual_seed(7))
    ms = timed(lambda: B.fold_perm(wk, perm_l2, H, d), reps=5)
    out["fold_perm"] = {"shape": [H * d, 4096], "ms": ms, "GB/s": 2 * wk.numel() * 2 / ms / 1e6}
    del calib, wk, wk_t
    k, v = W.make_kv(w, n_tokens=T, device=dev, batch=1)             # [1, 65536, 8, 128]
    z = torch.zeros(1, dtype=torch.int32, device=dev)
    ref = k[0, :4096, 0].float()
    rows = 2 * T * H
    fm = {}
    for n in (16, 32, 64):
        for p in (4, 6, 8):
            c = B.Cache(1, H, d, T, n, p, device=dev)
            B.append(c, k, v, z, perm_k=perm)
            ms = timed(lambda: B.append(c, k, v, z, perm_k=perm), reps=3)
            row_bytes = d * 2 + d * p // 8 + d // n
            mse_s = float(((B.dequant(c, "k", 0, 0, 0, 4096, perm=perm) - ref) ** 2).mean())
            B.append(c, k, None, z)
            mse_u = float(((B.dequant(c, "k", 0, 0, 0, 4096) - ref) ** 2).mean())
            fm[f"n{n}_p{p}"] = {"ms": ms, "GB/s": rows * row_bytes / ms / 1e6, "elements/s": rows * d / (ms * 1e-3),
                                "key_mse_unsorted": mse_u, "key_mse_ksort": mse_s}
            del c
    out["append"] = fm
    # read-back paths on the last cache: dequantisation of one head, rotation of rows in stored order
    c = B.Cache(1, H, d, T, 32, 4, device=dev)
    B.append(c, k, v, z, perm_k=perm)
    ms = timed(lambda: B.dequant(c, "k", 0, 0, 0, T, perm=perm), reps=5)
    out["dequant_one_head"] = {"tokens": T, "ms": ms, "GB/s": T * (68 + d * 4) / ms / 1e6}
    for name, dt, eb in (("f32", torch.float32, 4), ("bf16", torch.bfloat16, 2)):
        ms = timed(lambda: B.dequant_all(c, "k", T, perm=perm, out_dtype=dt), reps=5)
        out[f"dequant_all_heads_{name}"] = {"tokens": T, "heads": H, "ms": ms, "GB/s": T * H * (68 + d * eb) / ms / 1e6}
    ms = timed(lambda: B.dequant_all(c, "k", T), reps=5)
    out["dequant_all_heads_f32_stored_order"] = {"tokens": T, "heads": H, "ms": ms, "GB/s": T * H * (68 + d * 4) / ms / 1e6}
    _, perm_r, inv_r = B.calibrate(k[0, :4096].contiguous(), H, d)      # (a permutation together with ITS inverse)
    tabs = B.rope_tables(perm_r, inv_r, H, d, 10000.0, False, device=dev)
    rows = k[0]
    pos = torch.arange(T, dtype=torch.int32, device=dev)
    B.rope_apply(rows, pos, *tabs)
    ms = timed(lambda: B.rope_apply(rows, pos, *tabs), reps=5)
    out["rope_apply"] = {"rows": T * H, "ms": ms, "GB/s": 2 * rows.numel() * 2 / ms / 1e6}
    return out


def timed(fn, reps=1):
    """Milliseconds per call of fn(), CUDA events on the current stream."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def kernel_name(B, w, impl):
    if impl == B.DECODE_SIMT:
        return "decode_simt"
    if impl != B.DECODE_MMA_BF16 and w.mant_bits == 4:
        return "decode_mma4"
    if impl != B.DECODE_MMA_BF16 and w.mant_bits == 8 and w.block >= 32:
        return "decode_mma8"
    if impl != B.DECODE_MMA_BF16 and w.mant_bits == 6 and w.block >= 32 and w.n_q_heads == w.n_kv_heads:
        return "decode_mma6"
    return "decode_mma"


class StepRig:
    """One configuration made resident on the device: calibrated permutation, a cache prefilled with S - 1 tokens per
    sequence, the new token and the query of one decode step, output and workspace."""

    def __init__(self, B, w, dev, impl, rope=False, chunk=0):
        self.B, self.w, self.dev, self.impl, self.rope, self.chunk = B, w, dev, impl, rope, chunk
        S, Bn, Hkv, Hq, d = w.seq, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim
        self.es = 2 if w.dtype == "bf16" else 4
        self.calib = W.make_calibration(w, device=dev)
        _, self.perm_k, self.inv_perm_k = B.calibrate(self.calib, Hkv, d)
        self.kernel = kernel_name(B, w, impl)
        if rope:
            self.impl, self.kernel = B.DECODE_SIMT, "decode_simt_rope"
            self.rope_tabs = B.rope_tables(self.perm_k, self.inv_perm_k, Hkv, d, 10000.0, False, device=dev)
        self.cache = B.Cache(Bn, Hkv, d, S, w.block, w.mant_bits, device=dev)
        self.zeros = torch.zeros(Bn, dtype=torch.int32, device=dev)
        k, v = W.make_kv(w, n_tokens=S, device=dev)                      # [B, S, Hkv, d]
        self.k_pre, self.v_pre = k[:, :S - 1].contiguous(), v[:, :S - 1].contiguous()
        B.append(self.cache, self.k_pre, self.v_pre, self.zeros, perm_k=self.perm_k)
        self.k_new, self.v_new = k[:, S - 1:].contiguous(), v[:, S - 1:].contiguous()
        del k, v
        self.q = W.make_q(w, device=dev)
        self.start_pos = torch.full((Bn,), S - 1, dtype=torch.int32, device=dev)
        self.seq_lens = torch.full((Bn,), S, dtype=torch.int32, device=dev)
        self.out = torch.empty(Bn, Hq, d, dtype=torch.float32, device=dev)
        self.ws = torch.empty(B.decode_workspace_bytes(self.cache.fmt, Hq), dtype=torch.uint8, device=dev)
        torch.cuda.synchronize()

    def setup_timings(self):
        """Set-up calls of the path, timed once (not part of the step metric)."""
        B, w = self.B, self.w
        ex = {}
        ms = timed(lambda: B.calibrate(self.calib, w.n_kv_heads, w.head_dim), reps=3)
        ex["calibrate"] = {"tokens": int(self.calib.shape[0]), "ms": ms, "GB/s": self.calib.numel() * self.es / ms / 1e6}
        ms = timed(lambda: B.append(self.cache, self.k_pre, self.v_pre, self.zeros, perm_k=self.perm_k), reps=3)
        rows = 2 * w.batch * (w.seq - 1) * w.n_kv_heads
        row_bytes = w.head_dim * self.es + w.head_dim * w.mant_bits // 8 + w.head_dim // w.block
        ex["append_prefill"] = {"tokens_per_seq": w.seq - 1, "ms": ms, "GB/s": rows * row_bytes / ms / 1e6,
                                "elements/s": rows * w.head_dim / (ms * 1e-3)}
        return ex

    def free_setup(self):
        del self.calib, self.k_pre, self.v_pre
        self.calib = self.k_pre = self.v_pre = None

    def step(self):
        B, S = self.B, self.w.seq
        B.append(self.cache, self.k_new, self.v_new, self.start_pos, perm_k=self.perm_k)
        if self.rope:
            B.decode_attn_rope(self.cache, self.q, self.seq_lens, *self.rope_tabs, perm_k=self.perm_k, max_len_hint=S,
                               out=self.out, workspace=self.ws)
        else:
            B.decode_attn(self.cache, self.q, self.seq_lens, perm_k=self.perm_k, max_len_hint=S, impl=self.impl,
                          out=self.out, workspace=self.ws, chunk_tokens=self.chunk)

    def time_steps(self, steps, warmup, barrier):
        """-> (ms of `steps` steps, launches): the timed region of the step metric, nothing but the steps in it."""
        for _ in range(warmup):
            self.step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        launches0 = self.B.launch_count()
        e0.record()
        for _ in range(steps):
            self.step()
        e1.record()
        barrier()
        return e0.elapsed_time(e1), self.B.launch_count() - launches0

    def time_kernel(self, steps, warmup, barrier):
        """Mean duration (ms) of the main decode kernel over a second loop of the same steps, with a pair of CUDA
        events recorded around that kernel on its own stream.  Kept apart from the loop that times the step, so
        that the events sit in no step whose time is reported."""
        B = self.B
        kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in kev:              # an event gets its handle when it is first recorded
            a.record()
            b.record()
        for _ in range(warmup):
            self.step()
        barrier()
        for i in range(steps):
            B.profile_decode_events(*kev[i])
            self.step()
        B.profile_decode_events(None, None)
        barrier()
        return statistics.mean(a.elapsed_time(b) for a, b in kev)


def side_config(B, w, dev, impl, steps, warmup, local_rank, barrier):
    """A further configuration in the default run: the same step (append 1 token + decode attention), timed the same
    way, with its own clock sample.  -> dict for `extras`."""
    rig = StepRig(B, w, dev, impl)
    rig.free_setup()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    ms_total, _ = rig.time_steps(steps, warmup, barrier)
    kernel_ms = rig.time_kernel(min(steps, 200), 3, barrier)
    clocks = sampler.stop()
    flags = B.device_status()
    peak, _ = measured_peak()
    alg = decode_bytes(w)
    gbs = alg / (kernel_ms * 1e-3) / 1e9
    return {"workload": workload_name(w), "decode_kernel": rig.kernel, "steps": steps, "ms_per_step": ms_total / steps,
            "tokens/s": w.batch / (ms_total / steps * 1e-3), "kernel_ms": kernel_ms, "algorithmic_bytes": alg,
            "GB/s": gbs, "frac_of_measured_peak": gbs / peak, "device_status_flags": flags, "clocks": clocks}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, choices=[2, 3, 4])
    ap.add_argument("--decode-impl", default="auto", choices=["auto", "simt", "mma", "mma_bf16"])
    ap.add_argument("--ref-units", type=int, default=0, help="(batch, kv head) units per step of the reference arm (0 = sized for ~100 s)")
    ap.add_argument("--cpu-baseline-units", type=int, default=512)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (small cases for profiling)")
    ap.add_argument("--seq", type=int, default=0, help="override the cached sequence length")
    ap.add_argument("--q-heads", type=int, default=0, help="override the number of query heads (a multiple of the KV heads)")
    ap.add_argument("--mant-bits", type=int, default=0, choices=[0, 4, 6, 8])
    ap.add_argument("--block", type=int, default=0, choices=[0, 16, 32, 64, 128])
    ap.add_argument("--chunk", type=int, default=0, help="tokens per sequence chunk (0 = library default)")
    ap.add_argument("--rope", action="store_true", help="keys cached before the rotary embedding: time "
                    "kvbfp_decode_attn_rope (rotation after the read-back) instead; no end-to-end leg")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the set-up timings, the quality report and the further "
                    "configurations (GQA layer, mantissa sweep)")
    ap.add_argument("--sweep5", action="store_true", help="(kept for old command lines: the sweep is part of the default run)")
    ap.add_argument("--no-sweep5", action="store_true", help="skip the prefill/append and calibration sweep (8 KV heads, 65536 "
                    "new tokens, blocks 16/32/64 x mantissas 4/6/8, calibration over 2^20 tokens, read-back paths) in the extras")
    ap.add_argument("--sweep5-only", action="store_true", help="run that sweep alone and print its figures (a small case "
                    "for profiling the cache-write, calibration, read-back and rotation kernels)")
    args = ap.parse_args()
    w = W.CONFIGS[args.config]
    over = {k: v for k, v in (("batch", args.batch), ("seq", args.seq), ("mant_bits", args.mant_bits),
                              ("block", args.block), ("n_q_heads", args.q_heads)) if v}
    if over:
        w = dataclasses.replace(w, **over)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, w, rank)
        return

    if args.warmup < 3:
        args.warmup = 3
    from paper_2403_20137_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if args.sweep5_only:
        if rank == 0:
            print(json.dumps({"workload": "config5 sweep: 8 KV heads x 128, 65536 new bf16 tokens, calibration over 2^20 tokens",
                              "config5": sweep_config5(B, dev)}))
        return
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- set-up (untimed for the step metric): calibrate, prefill S-1 tokens ----------------------
    impl = {"auto": B.DECODE_AUTO, "simt": B.DECODE_SIMT, "mma": B.DECODE_MMA, "mma_bf16": B.DECODE_MMA_BF16}[args.decode_impl]
    S, Bn, Hkv, Hq, d = w.seq, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim
    rig = StepRig(B, w, dev, impl, rope=args.rope, chunk=args.chunk)
    if args.rope:
        args.no_e2e = True
    kernel, es = rig.kernel, rig.es
    extras = {}
    if not args.no_extras:
        extras.update(rig.setup_timings())
    rig.free_setup()

    # ---- device-resident timing: the step metric, then the main kernel's own duration ---------------
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ms_total, launches = rig.time_steps(args.steps, args.warmup, barrier)
    kernel_steps = min(args.steps, 500)
    kernel_ms = rig.time_kernel(kernel_steps, 3, barrier)
    flags = B.device_status()

    # ---- end to end: new token from pinned host memory, result back to the host, every step -------
    hk, hv, hq = rig.k_new.cpu().pin_memory(), rig.v_new.cpu().pin_memory(), rig.q.cpu().pin_memory()
    hout = torch.empty(Bn, Hq, d, dtype=torch.float32).pin_memory()
    staging = torch.empty(B.step_staging_bytes(rig.cache.fmt, Hq, rig.q.dtype), dtype=torch.uint8, device=dev)

    step_host = B.HostStep(rig.cache, hk, hv, hq, rig.start_pos, rig.seq_lens, hout, staging, rig.ws, perm_k=rig.perm_k,
                           max_len_hint=S, impl=rig.impl)       # the arguments of the loop's call, marshalled once

    n_e2e = 0 if args.no_e2e else args.steps
    for _ in range(args.warmup if n_e2e else 0):
        step_host()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(n_e2e):
        step_host()
    f1.record()
    barrier()
    ms_e2e = f0.elapsed_time(f1) if n_e2e else float("nan")
    clocks = sampler.stop() if rank == 0 else None
    e2e_ok = bool(torch.equal(hout.to(dev), rig.out)) if n_e2e else None

    # ---- max over ranks -----------------------------------------------------------------------------
    ms_total, ms_e2e, kernel_ms = max_over_ranks([ms_total, ms_e2e, kernel_ms], dist, dev)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- further configurations and the quality report (rank 0, outside every timed region above) ---
    if not args.no_extras and world == 1 and not over and args.config == 3 and impl == B.DECODE_AUTO and not args.rope:
        extras["config4"] = side_config(B, W.CONFIGS[4], dev, impl, 300, 10, local_rank, barrier)
        extras["mant_sweep"] = {f"p{p}": side_config(B, dataclasses.replace(w, mant_bits=p), dev, impl, 300, 10,
                                                     local_rank, barrier) for p in (6, 8)}
    if not args.no_extras and world == 1 and not args.no_sweep5 and not over and args.config == 3:
        extras["config5"] = sweep_config5(B, dev)
    if not args.no_extras and world == 1:
        from paper_2403_20137_b200 import quality as Q
        nq = max(16, min(2048, S // 16 * 16))
        extras["quality"] = Q.quality_report(w, dev, n_tokens=nq)
        extras["quality_outliers_in_v"] = Q.quality_report(w, dev, n_tokens=nq, outliers_in_v=True, sort_v=True)

    ms_step = ms_total / args.steps
    value = whole_job_throughput(Bn, world, ms_step)
    e2e_value = whole_job_throughput(Bn, world, ms_e2e / args.steps) if n_e2e else None
    peak, peak_src = measured_peak()
    alg = decode_bytes(w)
    achieved = alg / (kernel_ms * 1e-3) / 1e9
    h2d = 2 * Bn * Hkv * d * es + Bn * Hq * d * es
    d2h = Bn * Hq * d * 4

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16" if kernel in ("decode_mma4", "decode_mma8", "decode_mma6") else ("bf16" if kernel == "decode_mma" else "f32"),
        "data": "synthetic",
        "config": config_of(w),
        "details": {"per_gpu_batch": Bn, "decode_kernel": kernel, "device_status_flags": flags,
                    "e2e_matches_device_path": e2e_ok, "tokens_per_s_if_32_layers": value / 32.0},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": (ms_e2e / args.steps) if n_e2e else None},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic_per_launch(kernel, w),
                     "algorithmic_bytes": alg, "kernel_ms": kernel_ms, "peak_source": peak_src,
                     "kernel_timing": f"CUDA events around the main kernel, on its stream, in a loop of {kernel_steps} steps "
                                      "of its own right after the loop that times the step; the event records keep "
                                      "the kernel from overlapping its launch with the kernel before it, which the "
                                      "step loop does (programmatic stream serialization), so this figure contains "
                                      "a few microseconds of launch latency that the step does not pay",
                     "frac_of_nominal_8000_GBs": achieved / 8000.0},
        "extras": extras or None,
    }
    if not args.no_cpu_baseline and world == 1:
        sample = min(args.cpu_baseline_units, Bn * Hkv)
        ost = OracleStep(w, sample)
        reps = 2
        t = statistics.mean(ost.run() for _ in range(reps))
        t_full = t * (Bn * Hkv) / sample
        result["cpu_baseline"] = {
            "value": Bn / t_full, "unit": UNIT, "cores": ost.cores, "kind": "oracle",
            "sample": (f"{sample} of {Bn * Hkv} (batch, kv head) units of one step, {reps} repetitions of {t:.2f} s on "
                       f"{ost.cores} threads, scaled to the full step")}
    else:
        result["cpu_baseline"] = None
    print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
