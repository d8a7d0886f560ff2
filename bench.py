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


def workload_name(w):
    return (f"config{w.config}: B{w.batch} Hq{w.n_q_heads} Hkv{w.n_kv_heads} d{w.head_dim} S{w.seq} {w.dtype} "
            f"BFP block{w.block} mant{w.mant_bits}; append 1 token/seq + decode attention")


def decode_bytes(w):
    """Algorithmic bytes of one decode launch: packed K and V rows of every cached token, once."""
    row = w.head_dim * w.mant_bits // 8 + w.head_dim // w.block
    return 2 * row * w.batch * w.n_kv_heads * w.seq


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy bandwidth)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier copy measurement on this pool)"


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
        "config": {"workload": workload_name(w)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": st.cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, choices=[2, 3, 4])
    ap.add_argument("--decode-impl", default="auto", choices=["auto", "simt", "mma"])
    ap.add_argument("--ref-units", type=int, default=0, help="(batch, kv head) units per step of the reference arm (0 = sized for ~100 s)")
    ap.add_argument("--cpu-baseline-units", type=int, default=256)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (small cases for profiling)")
    ap.add_argument("--seq", type=int, default=0, help="override the cached sequence length")
    ap.add_argument("--mant-bits", type=int, default=0, choices=[0, 4, 6, 8])
    ap.add_argument("--block", type=int, default=0, choices=[0, 16, 32, 64, 128])
    ap.add_argument("--chunk", type=int, default=0, help="tokens per sequence chunk (0 = library default)")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    w = W.CONFIGS[args.config]
    import dataclasses
    over = {k: v for k, v in (("batch", args.batch), ("seq", args.seq), ("mant_bits", args.mant_bits),
                              ("block", args.block)) if v}
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
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # ---- set-up (untimed): calibrate, prefill S-1 tokens -----------------------------------------
    impl = {"auto": B.DECODE_AUTO, "simt": B.DECODE_SIMT, "mma": B.DECODE_MMA}[args.decode_impl]
    S, Bn, Hkv, Hq, d = w.seq, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim
    calib = W.make_calibration(w, device=dev)
    _, perm_k, _ = B.calibrate(calib, Hkv, d)
    del calib
    cache = B.Cache(Bn, Hkv, d, S, w.block, w.mant_bits, device=dev)
    zeros = torch.zeros(Bn, dtype=torch.int32, device=dev)
    k, v = W.make_kv(w, n_tokens=S, device=dev)                      # [B, S, Hkv, d]
    B.append(cache, k[:, :S - 1].contiguous(), v[:, :S - 1].contiguous(), zeros, perm_k=perm_k)
    k_new, v_new = k[:, S - 1:].contiguous(), v[:, S - 1:].contiguous()
    del k, v
    q = W.make_q(w, device=dev)
    start_pos = torch.full((Bn,), S - 1, dtype=torch.int32, device=dev)
    seq_lens = torch.full((Bn,), S, dtype=torch.int32, device=dev)
    out = torch.empty(Bn, Hq, d, dtype=torch.float32, device=dev)
    ws = torch.empty(B.decode_workspace_bytes(cache.fmt, Hq), dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()

    def step():
        B.append(cache, k_new, v_new, start_pos, perm_k=perm_k)
        B.decode_attn(cache, q, seq_lens, perm_k=perm_k, max_len_hint=S, impl=impl, out=out, workspace=ws,
                      chunk_tokens=args.chunk)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing -------------------------------------------------------------------
    for _ in range(args.warmup):
        step()
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in kev:              # an event gets its handle when it is first recorded
        a.record()
        b.record()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    launches0 = B.launch_count()
    e0.record()
    for i in range(args.steps):
        B.profile_decode_events(*kev[i])
        step()
    e1.record()
    barrier()
    launches = B.launch_count() - launches0
    B.profile_decode_events(None, None)
    ms_total = e0.elapsed_time(e1)
    kernel_ms = statistics.mean(a.elapsed_time(b) for a, b in kev)
    flags = B.device_status()

    # ---- end to end: new token from pinned host memory, result back to the host, every step -------
    hk, hv, hq = k_new.cpu().pin_memory(), v_new.cpu().pin_memory(), q.cpu().pin_memory()
    hout = torch.empty(Bn, Hq, d, dtype=torch.float32).pin_memory()
    staging = torch.empty(B.step_staging_bytes(cache.fmt, Hq, q.dtype), dtype=torch.uint8, device=dev)

    def step_host():
        B.decode_step_host(cache, hk, hv, hq, start_pos, seq_lens, hout, staging, ws, perm_k=perm_k, max_len_hint=S,
                           impl=impl)

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
    e2e_ok = bool(torch.equal(hout.to(dev), out)) if n_e2e else None

    # ---- max over ranks -----------------------------------------------------------------------------
    if dist is not None:
        t = torch.tensor([ms_total, ms_e2e, kernel_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total, ms_e2e, kernel_ms = t.tolist()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_step = ms_total / args.steps
    value = world * Bn / (ms_step * 1e-3)
    e2e_value = world * Bn / (ms_e2e / args.steps * 1e-3)
    peak, peak_src = measured_peak()
    alg = decode_bytes(w)
    achieved = alg / (kernel_ms * 1e-3) / 1e9
    es = 2 if w.dtype == "bf16" else 4
    h2d = 2 * Bn * Hkv * d * es + Bn * Hq * d * es
    d2h = Bn * Hq * d * 4

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(w), "per_gpu_batch": Bn, "decode_kernel": args.decode_impl,
                   "l2": f"inputs larger than L2: {alg / 1e6:.0f} MB of cache read per step vs 126 MB L2",
                   "device_status_flags": flags, "e2e_matches_device_path": e2e_ok},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode_mma" if impl != B.DECODE_SIMT else "decode_simt",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "algorithmic_bytes": alg, "kernel_ms": kernel_ms, "peak_source": peak_src},
    }
    if not args.no_cpu_baseline and world == 1:
        sample = min(args.cpu_baseline_units, Bn * Hkv)
        ost = OracleStep(w, sample)
        t, cores = ost.run(), ost.cores
        t_full = t * (Bn * Hkv) / sample
        result["cpu_baseline"] = {
            "value": Bn / t_full, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{sample} of {Bn * Hkv} (batch, kv head) units of one step, {t:.1f} s, scaled to the full step"}
    else:
        result["cpu_baseline"] = None
    print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
