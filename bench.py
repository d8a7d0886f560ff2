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

# DRAM traffic of the dominant kernel from one ncu capture (profiles/decode_mma4_b4_s8192_ncu_full.md; the 8-bit
# kernel: profiles/other_decode_kernels_b4_s8192_ncu_sections.md):
# dram__bytes_read.sum + dram__bytes_write.sum per (batch, kv head, token) unit on a smaller case of the
# same kernel, scaled by the units of a launch.  Valid only while the kernel sources still hash to the
# value recorded with the capture; otherwise the bench reports null.
TRAFFIC = {"decode_mma4": {"bytes_per_unit": 139.7314, "block": 32, "mant_bits": 4, "sources_sha256": "1f77fe48622022daf80f46a8ff271438062c3f8d00a14cd609cbd42127c1b2a5"},
           "decode_mma8": {"bytes_per_unit": 264.3372, "block": 32, "mant_bits": 8, "sources_sha256": "0e0ae313fe6df113eeef12d6dc9031be944ef871e159f7e0f2dd54418cc1c5ce"}}
KERNEL_SOURCES = {"decode_mma4": ["paper_2403_20137_b200/csrc/decode_mma4.cu", "paper_2403_20137_b200/csrc/ptx.cuh"],
                  "decode_mma8": ["paper_2403_20137_b200/csrc/decode_mma8.cu", "paper_2403_20137_b200/csrc/ptx.cuh"]}


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
        "config": {"workload": workload_name(w)},
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
    _, _, inv = B.calibrate(k[0, :4096].contiguous(), H, d)
    tabs = B.rope_tables(perm, inv, H, d, 10000.0, False, device=dev)
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
                    "kvbfp_decode_attn_rope (fp32 kernel, rotation after the read-back) instead; no end-to-end leg")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the set-up timings and the quality report")
    ap.add_argument("--sweep5", action="store_true", help="add the prefill/append and calibration sweep (8 KV heads, 65536 new\n                    tokens, blocks 16/32/64 x mantissas 4/6/8, calibration over 2^20 tokens) to the extras")
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
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # ---- set-up (untimed for the step metric): calibrate, prefill S-1 tokens ----------------------
    impl = {"auto": B.DECODE_AUTO, "simt": B.DECODE_SIMT, "mma": B.DECODE_MMA, "mma_bf16": B.DECODE_MMA_BF16}[args.decode_impl]
    kernel = "decode_simt" if impl == B.DECODE_SIMT else \
        ("decode_mma4" if (w.mant_bits == 4 and impl != B.DECODE_MMA_BF16) else
         "decode_mma8" if (w.mant_bits == 8 and w.block >= 32 and impl != B.DECODE_MMA_BF16) else "decode_mma")
    S, Bn, Hkv, Hq, d = w.seq, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim
    es = 2 if w.dtype == "bf16" else 4
    extras = {}
    calib = W.make_calibration(w, device=dev)
    _, perm_k, inv_perm_k = B.calibrate(calib, Hkv, d)
    if args.rope:
        impl, kernel, args.no_e2e = B.DECODE_SIMT, "decode_simt_rope", True
        rope_tabs = B.rope_tables(perm_k, inv_perm_k, Hkv, d, 10000.0, False, device=dev)
    if not args.no_extras:
        ms = timed(lambda: B.calibrate(calib, Hkv, d), reps=3)
        extras["calibrate"] = {"tokens": int(calib.shape[0]), "ms": ms, "GB/s": calib.numel() * es / ms / 1e6}
    del calib
    cache = B.Cache(Bn, Hkv, d, S, w.block, w.mant_bits, device=dev)
    zeros = torch.zeros(Bn, dtype=torch.int32, device=dev)
    k, v = W.make_kv(w, n_tokens=S, device=dev)                      # [B, S, Hkv, d]
    k_pre, v_pre = k[:, :S - 1].contiguous(), v[:, :S - 1].contiguous()
    B.append(cache, k_pre, v_pre, zeros, perm_k=perm_k)
    if not args.no_extras:
        ms = timed(lambda: B.append(cache, k_pre, v_pre, zeros, perm_k=perm_k), reps=3)
        rows = 2 * Bn * (S - 1) * Hkv
        row_bytes = d * es + d * w.mant_bits // 8 + d // w.block
        extras["append_prefill"] = {"tokens_per_seq": S - 1, "ms": ms, "GB/s": rows * row_bytes / ms / 1e6,
                                    "elements/s": rows * d / (ms * 1e-3)}
        # quality on one head: key MSE and pre-softmax score error with and without K-sort (Table I's direction)
        Tq = max(16, min(4096, (S - 1) // 16 * 16))
        plain = B.Cache(1, Hkv, d, Tq, w.block, w.mant_bits, device=dev)
        sortd = B.Cache(1, Hkv, d, Tq, w.block, w.mant_bits, device=dev)
        z1 = torch.zeros(1, dtype=torch.int32, device=dev)
        kk = k[:1, :Tq].contiguous()
        B.append(plain, kk, None, z1)
        B.append(sortd, kk, None, z1, perm_k=perm_k)
        ref = kk[0, :, 0].float()
        dq_p = B.dequant(plain, "k", 0, 0, 0, Tq)
        dq_s = B.dequant(sortd, "k", 0, 0, 0, Tq, perm=perm_k)
        qv = W.make_q(w, device=dev)[0, 0].float()
        s_ref = ref @ qv
        extras["quality_head0"] = {
            "bits_per_element": w.mant_bits + 8.0 / w.block,
            "key_mse_unsorted": float(((dq_p - ref) ** 2).mean()), "key_mse_ksort": float(((dq_s - ref) ** 2).mean()),
            "score_rms_err_unsorted": float(((dq_p @ qv - s_ref) ** 2).mean().sqrt()),
            "score_rms_err_ksort": float(((dq_s @ qv - s_ref) ** 2).mean().sqrt())}
        del plain, sortd, kk, dq_p, dq_s
    k_new, v_new = k[:, S - 1:].contiguous(), v[:, S - 1:].contiguous()
    del k, v, k_pre, v_pre
    if args.sweep5 and rank == 0:
        extras["config5"] = sweep_config5(B, dev)
    q = W.make_q(w, device=dev)
    start_pos = torch.full((Bn,), S - 1, dtype=torch.int32, device=dev)
    seq_lens = torch.full((Bn,), S, dtype=torch.int32, device=dev)
    out = torch.empty(Bn, Hq, d, dtype=torch.float32, device=dev)
    ws = torch.empty(B.decode_workspace_bytes(cache.fmt, Hq), dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()

    def step():
        B.append(cache, k_new, v_new, start_pos, perm_k=perm_k)
        if args.rope:
            B.decode_attn_rope(cache, q, seq_lens, *rope_tabs, perm_k=perm_k, max_len_hint=S, out=out, workspace=ws)
        else:
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
    ms_total, ms_e2e, kernel_ms = max_over_ranks([ms_total, ms_e2e, kernel_ms], dist, dev)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

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
        "dtype": "f16" if kernel in ("decode_mma4", "decode_mma8") else ("bf16" if kernel == "decode_mma" else "f32"),
        "data": "synthetic",
        "config": {"workload": workload_name(w), "per_gpu_batch": Bn, "decode_kernel": kernel,
                   "l2": f"inputs larger than L2: {alg / 1e6:.0f} MB of cache read per step vs 126 MB L2",
                   "device_status_flags": flags, "e2e_matches_device_path": e2e_ok,
                   "tokens_per_s_if_32_layers": value / 32.0},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": (ms_e2e / args.steps) if n_e2e else None},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic_per_launch(kernel, w),
                     "algorithmic_bytes": alg, "kernel_ms": kernel_ms, "peak_source": peak_src,
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
