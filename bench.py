#!/usr/bin/env python
"""Benchmark of the fused eviction path (score + select + compact) on synthetic Llama-3.1-8B-shaped inputs.

One step = one call of restkv_evict over one layer of the long-context workload (batch 1, 32 query / 8 KV
heads, head_dim 128, n = 131072 prefix rows, window 32, budget 2048, bf16).  Metric: prefix tokens scored and
evicted per second per layer.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg4]

N > 1 (under torchrun): every rank runs an independent replica of the layer on its own GPU -- the path has no
exchange step, so there is no data-path collective; NCCL is used only for the barrier and the max over ranks.
`--impl reference` times the CPU oracle (test infrastructure) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "prefix tokens/sec scored+evicted per layer at 128k"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 256 << 20


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


def algorithmic_bytes(case, keep):
    """K and V read once plus the compacted cache written (bytes per step)."""
    es = 2 if case.dtype == "bf16" else 4
    kv = 2 * case.batch * case.n_kv_heads * case.n_kv * case.head_dim * es
    out = 2 * case.batch * case.n_kv_heads * keep * case.head_dim * es
    return kv, out


def algorithmic_flops(case):
    """Three dense contractions per prefix token and KV head: Q K^T, P V, V O^T."""
    R = case.w * case.group
    return 3 * 2 * R * case.head_dim * case.batch * case.n_kv_heads * case.n


def max_over_ranks(total_ms, world, device):
    """The slowest rank's time for the timed region (the job ends when the last replica ends)."""
    if world <= 1:
        return float(total_ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([total_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank_step, world, steps, total_ms):
    """Prefix tokens per second over all replicas: every rank processes its own layer in every step."""
    return world * tokens_per_rank_step * steps / (total_ms / 1e3)


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel, from an ncu capture
# of this workload, together with the digest of the kernel sources the capture was taken on: the figure is reported
# only while those sources are unchanged, otherwise `traffic` is null.
KERNEL_TRAFFIC = {"cfg4": {"bytes": 1024809984 + 27120896, "sources_sha256": "c2a2d5d570c4642c49dda616763660c7e2819fce2c4e152d8a36ee85e09c58ec"}}
KERNEL_SOURCES = ("tc_fused.cu", "tc_common.cuh", "sm100_ptx.cuh")


def kernel_sources_digest():
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2605_08840_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_traffic(workload):
    rec = KERNEL_TRAFFIC.get(workload)
    if not rec or rec["bytes"] is None or rec["sources_sha256"] != kernel_sources_digest():
        return None
    return rec["bytes"]


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons while the timed region runs.

    NVML is polled in-process every ~2 ms (the timed region lasts a few milliseconds, too short for
    `nvidia-smi -lms`); if the NVML binding is missing, one `nvidia-smi` query at the end stands in.  Read-only."""
    REASONS = (("hw_slowdown", 0x8), ("sw_power_cap", 0x4), ("sw_thermal_slowdown", 0x20),
               ("hw_thermal_slowdown", 0x40))

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.sm, self.bits = [], 0
        self.max_mhz = None
        self.thread = None
        self.stop_flag = False
        self.nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            index = self.gpu
            if visible:
                entry = visible.split(",")[self.gpu].strip()
                index = int(entry) if entry.isdigit() else self.gpu
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
        except Exception:
            self.nvml = None
            return
        self.thread = threading.Thread(target=self._poll, daemon=True)
        self.thread.start()

    def _poll(self):
        nv = self.nvml
        while not self.stop_flag:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                self.bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
            except Exception:
                break
            time.sleep(0.001)

    def stop(self):
        if self.nvml is None:
            return self._smi_once()
        self.stop_flag = True
        self.thread.join(timeout=2)
        sm = sorted(self.sm)
        reasons = sorted(name for name, bit in self.REASONS if self.bits & bit)
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(sm), "source": "nvml, 1 ms polling during the timed steps and the per-kernel passes"}

    def _smi_once(self):
        fields = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
                  "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            out = subprocess.run(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + fields,
                                  "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
            parts = [x.strip() for x in out.strip().splitlines()[0].split(",")]
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            reasons = sorted(n for n, v in zip(names, parts[2:6]) if v.lower().startswith("active"))
            return {"sm_mhz": float(parts[0]), "sm_max_mhz": float(parts[1]), "reasons": reasons, "samples": 1,
                    "source": "nvidia-smi, one query after the timed region"}
        except Exception:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clock query unavailable"], "samples": 0}


# ------------------------------------------------------------------------------------------------
def time_oracle(inp, heads, budget, repeats=1):
    """Wall time of the oracle's score + select + compact on the given KV heads of the workload."""
    import numpy as np
    import oracle
    c = inp.case
    G = c.group
    qh = np.concatenate([np.arange(h * G, (h + 1) * G) for h in heads])
    Q, K, V = (np.ascontiguousarray(x) for x in (inp.Q[:, qh], inp.K[:, heads], inp.V[:, heads]))
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        res = oracle.score(Q, K, V, causal_tail=c.causal_tail, ema_decay=c.ema_decay, width=c.width, shift=c.shift,
                           want_I_hat=False)
        idx = oracle.select(res.scores, budget)
        oracle.compact(K, idx)
        oracle.compact(V, idx)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best


def cpu_baseline(inp, budget, target_seconds=12.0):
    """The oracle as it stands on the host cores, on a bounded sample: whole KV heads of the workload."""
    import oracle
    c = inp.case
    t1 = time_oracle(inp, [0], budget)
    heads = max(1, min(c.n_kv_heads, int(target_seconds / 3.0 / max(t1, 1e-3))))
    t = time_oracle(inp, list(range(heads)), budget, repeats=3)     # best of three: the host is shared
    tokens = c.batch * c.n * heads / c.n_kv_heads     # layer-equivalent prefix tokens in the sample
    return {"value": tokens / t, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "%d of %d KV heads of the workload at full length n=%d (score+select+compact), best of 3: %.2f s"
                      % (heads, c.n_kv_heads, c.n, t)}


def run_reference(args, case):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2605_08840_b200.inputs import make_inputs
    inp = make_inputs(case)
    budget = case.budget
    t1 = time_oracle(inp, [0], budget)
    per_step_budget = 150.0 / max(1, args.steps + args.warmup)
    heads = max(1, min(case.n_kv_heads, int(per_step_budget / max(t1, 1e-3))))
    sel = list(range(heads))
    for _ in range(args.warmup):
        time_oracle(inp, sel, budget)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time_oracle(inp, sel, budget)
    dt = (time.perf_counter() - t0) / args.steps
    tokens = case.batch * case.n * heads / case.n_kv_heads
    value = tokens / dt
    sample = "%d of %d KV heads at full length n=%d per step" % (heads, case.n_kv_heads, case.n)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(case, l2="n/a (CPU)"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(case, l2):
    return {"workload": "%s: one layer, batch %d, %d query / %d KV heads, head_dim %d, n=%d prefix rows, window %d, "
                        "budget %d, pool width %d, ema_decay %.2f, %s, planted heavy hitters + sinks"
                        % (case.name, case.batch, case.n_q_heads, case.n_kv_heads, case.head_dim, case.n, case.w,
                           case.budget, case.width, case.ema_decay, case.dtype),
            "global_batch": case.batch, "seq_len": case.n, "parallelism": "replicas", "l2": l2}


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the timings beside the headline that came with the variants, the adaptive window, "
                         "re-eviction and the output projection (short runs under a profiler)")
    ap.add_argument("--path", type=int, default=0, help="0 auto, 1 force SIMT, 2 require tensor cores")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2605_08840_b200.inputs import CONFIGS, make_inputs
    case = CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, case)
        return

    import numpy as np
    import torch
    from paper_2605_08840_b200 import binding as rk

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank: an independent replica of the layer (per-rank seed so the replicas are not identical)
    inp = make_inputs(case, seed=case.seed + 1000 * rank)
    q_np, k_np, v_np = inp.device_arrays()
    tdt = torch.bfloat16 if case.dtype == "bf16" else torch.float32

    def dev(a):
        t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
        return t.view(tdt) if case.dtype == "bf16" else t

    Q, K, V = dev(q_np), dev(k_np), dev(v_np)
    handle = rk.Handle()
    handle.set_kernel_path(args.path)
    shape = rk.make_shape(case.batch, case.n_q_heads, case.n_kv_heads, case.head_dim, case.n_kv, case.w,
                          case.causal_tail, rk.BF16 if case.dtype == "bf16" else rk.F32)
    pool = rk.fixed_pool(case.width, case.shift)
    keep = min(case.budget, case.n_kv)
    BH = (case.batch, case.n_kv_heads)
    indices = torch.empty(BH + (keep,), dtype=torch.int32, device="cuda")
    K_out = torch.empty(BH + (keep, case.head_dim), dtype=tdt, device="cuda")
    V_out = torch.empty_like(K_out)
    ws = torch.empty(handle.workspace_bytes(shape, case.budget), dtype=torch.uint8, device="cuda")
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    def step():
        handle.evict(shape, Q, K, V, case.ema_decay, pool, case.budget, indices, K_out, V_out, ws)

    for _ in range(args.warmup):
        flush.zero_()
        step()
    barrier()
    fused = handle.last_evict_fused_select()
    launches0 = handle.launch_count()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    step_ms = []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(args.steps):
        flush.zero_()                       # evict the previous step's lines from L2 (not timed)
        ev0.record()
        step()
        ev1.record()
        torch.cuda.synchronize()
        step_ms.append(ev0.elapsed_time(ev1))
    barrier()
    launches = handle.launch_count() - launches0

    # Per-kernel durations in passes of their own (the event records between the launches would sit inside the
    # timed region otherwise): CUDA events recorded by the library right around each launch, on the call's stream.
    # On the tensor-core path with a fixed window one persistent launch does everything (pass 1, merge, pass 2,
    # pooling, selection, gather); a second pass with the selection as its own kernel gives the split.
    def kernel_pass(kernel_ids, reps):
        prof = {}
        for name in kernel_ids:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); b.record()
            prof[name] = (a, b)
        torch.cuda.synchronize()
        for name, kid in kernel_ids.items():
            handle.set_profile_events(kid, *prof[name])
        ms = {k: [] for k in kernel_ids}
        for _ in range(reps):
            flush.zero_()
            step()
            torch.cuda.synchronize()
            for name in kernel_ids:
                ms[name].append(prof[name][0].elapsed_time(prof[name][1]))
        for kid in kernel_ids.values():
            handle.set_profile_events(kid, None, None)
        return {k: float(np.mean(v)) for k, v in ms.items()}

    split_ids = {"score": rk.KERNEL_PASS2, "pool_select_compact": rk.KERNEL_SELECT}
    if case.batch * case.n_kv_heads * 8 > 148:      # many rows: the gather runs as its own kernel
        split_ids = {"score": rk.KERNEL_PASS2, "pool_select": rk.KERNEL_SELECT, "compact": rk.KERNEL_COMPACT}
    reps = max(3, min(args.steps, 20))
    kmean_split = None
    if fused:
        kmean = kernel_pass({"score_pool_select_compact": rk.KERNEL_PASS2}, reps)
        handle.set_fused_select(False)
        kmean_split = kernel_pass(split_ids, reps)
        handle.set_fused_select(True)
    else:
        kmean = kernel_pass(split_ids, reps)
    clocks = sampler.stop() if rank == 0 else None      # sampled through the timed steps and the per-kernel passes
    assert handle.poll_status() == rk.RESTKV_OK

    total_ms = max_over_ranks(float(sum(step_ms)), world, "cuda")
    tokens_per_step = world * case.batch * case.n
    value = whole_job_value(case.batch * case.n, world, args.steps, total_ms)
    ms_per_step = total_ms / args.steps

    # ---- one decode step over the compacted cache and over the full cache (context for the paper's 10.61x) ----
    decode = None
    if rank == 0:
        from paper_2605_08840_b200.inputs import make_decode_query, round_to_bf16_bits
        q_np2 = make_decode_query(inp)                 # seeded
        qd = dev(round_to_bf16_bits(q_np2).view(np.int16) if case.dtype == "bf16" else q_np2)
        dout = torch.empty(case.batch, case.n_q_heads, case.head_dim, dtype=torch.float32, device="cuda")

        def time_decode(Kc, Vc, rows):
            for _ in range(3):
                handle.decode(shape, qd, Kc, Vc, rows, dout, ws)
            ts = []
            for _ in range(10):
                flush.zero_()
                ev0.record()
                handle.decode(shape, qd, Kc, Vc, rows, dout, ws)
                ev1.record()
                torch.cuda.synchronize()
                ts.append(ev0.elapsed_time(ev1))
            return float(np.median(ts)) * 1e3
        us_c = time_decode(K_out, V_out, keep)
        us_f = time_decode(K, V, case.n_kv)
        row_bytes = 2 * case.batch * case.n_kv_heads * case.head_dim * (2 if case.dtype == "bf16" else 4)
        decode = {"compact_us": us_c, "full_us": us_f, "ratio": us_f / us_c, "rows_compact": keep,
                  "rows_full": case.n_kv, "compact_gbs": row_bytes * keep / us_c / 1e3,
                  "full_gbs": row_bytes * case.n_kv / us_f / 1e3, "note": "one layer, one token, this kernel only; the paper's 10.61x is the "
                  "whole model's per-token latency on an A800 with FlashAttention-2"}

    # ---- scores from given window outputs and log-sum-exps (what a prefill has at hand): one read of K and V ----
    from_lse = None
    if rank == 0 and case.causal_tail == 0:
        G, w, d = case.group, case.w, case.head_dim
        scale = 1.0 / float(np.sqrt(d))
        O_obs = torch.empty(case.batch, case.n_q_heads, w, d, dtype=torch.float32, device="cuda")
        L_obs = torch.empty(case.batch, case.n_q_heads, w, dtype=torch.float32, device="cuda")
        for bi in range(case.batch):          # the window rows' attention, as the prefill would have left it (not timed)
            for h in range(case.n_kv_heads):
                qf = Q[bi, h * G:(h + 1) * G].float().reshape(G * w, d)
                sc = scale * (qf @ K[bi, h].float().T)
                lse = torch.logsumexp(sc, dim=-1)
                O_obs[bi, h * G:(h + 1) * G] = (torch.exp(sc - lse[:, None]) @ V[bi, h].float()).view(G, w, d)
                L_obs[bi, h * G:(h + 1) * G] = lse.view(G, w)
                del sc
        sc_out = torch.empty(BH + (case.n_kv,), dtype=torch.float32, device="cuda")
        for _ in range(3):
            handle.score_from_lse(shape, Q, K, V, O_obs, L_obs, case.ema_decay, pool, sc_out, ws)
        ts = []
        for _ in range(10):
            flush.zero_()
            ev0.record()
            handle.score_from_lse(shape, Q, K, V, O_obs, L_obs, case.ema_decay, pool, sc_out, ws)
            ev1.record()
            torch.cuda.synchronize()
            ts.append(ev0.elapsed_time(ev1))
        assert handle.poll_status() == rk.RESTKV_OK
        ms_l = float(np.median(ts))
        te = []
        for it in range(13):
            flush.zero_()
            ev0.record()
            handle.evict_from_lse(shape, Q, K, V, O_obs, L_obs, case.ema_decay, pool, case.budget, indices, K_out,
                                  V_out, ws)
            ev1.record()
            torch.cuda.synchronize()
            if it >= 3:
                te.append(ev0.elapsed_time(ev1))
        assert handle.poll_status() == rk.RESTKV_OK
        ms_e = float(np.median(te))
        kv_b, out_b = algorithmic_bytes(case, keep)
        pk = load_peaks()
        t_roof = max((kv_b + out_b) / (pk["hbm_gbs"] * 1e9), algorithmic_flops(case) * 2.0 / 3.0 / (pk["bf16_tflops"] * 1e12)) * 1e3
        from_lse = {"note": "the window rows' O and log-sum-exp given (as after prompt prefilling): K and V read once; "
                            "beside the headline, not instead of it",
                    "score_from_lse_ms": ms_l, "score_tokens_per_s": case.batch * case.n / (ms_l * 1e-3),
                    "score_hbm_frac": kv_b / (ms_l * 1e-3) / 1e9 / pk["hbm_gbs"],
                    "evict_from_lse_ms": ms_e, "evict_tokens_per_s": case.batch * case.n / (ms_e * 1e-3),
                    "evict_path_roofline_frac": t_roof / ms_e, "t_roof_ms": t_roof,
                    "roofline_note": "max(bytes / HBM peak, flops / bf16 peak): K, V once + compacted write; two "
                                     "contractions (Q K^T, V O^T) instead of three"}
        del O_obs, L_obs, sc_out

    # ---- the ablation variants of Appendix G as modes of the same path (beside the headline) ----
    variants = None
    if rank == 0 and world == 1 and not args.no_extras:
        labelled = (("attention_weight__mean_over_window", (rk.INDICATOR_ATTENTION, rk.TEMPORAL_MEAN, 0, 0)),
                    ("attention_weight_times_value_norm__ema", (rk.INDICATOR_ATTENTION_VNORM, rk.TEMPORAL_EMA, 0, 0)),
                    ("reconstruction__inverted_ema__max_pool__group_max",
                     (rk.INDICATOR_RECONSTRUCTION, rk.TEMPORAL_INV_EMA, rk.SPATIAL_MAX, rk.GROUP_MAX)))
        variants = {"note": "restkv_evict under restkv_set_variant, same workload and timing as the headline step",
                    "evict_ms": {}}
        for label, v in labelled:
            handle.set_variant(*v)
            try:
                tv = []
                for it in range(11):
                    flush.zero_()
                    ev0.record()
                    step()
                    ev1.record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        tv.append(ev0.elapsed_time(ev1))
            finally:
                handle.set_variant()
            assert handle.poll_status() == rk.RESTKV_OK
            variants["evict_ms"][label] = float(np.median(tv))

    # ---- the adaptive window of Eq. 10-12 (per-query top-B of the raw indicator, D_front / D_rear) ----
    adaptive = None
    if rank == 0 and world == 1 and not args.no_extras:
        apool = rk.adaptive_pool(2000.0, case.width, case.budget)
        ws_a = torch.empty(handle.workspace_bytes(shape, case.budget, adaptive=True), dtype=torch.uint8, device="cuda")

        def time_adaptive(path, reps):
            handle.set_kernel_path(path)
            try:
                ta = []
                for it in range(reps + 2):
                    flush.zero_()
                    ev0.record()
                    handle.evict(shape, Q, K, V, case.ema_decay, apool, case.budget, indices, K_out, V_out, ws_a)
                    ev1.record()
                    torch.cuda.synchronize()
                    if it >= 2:
                        ta.append(ev0.elapsed_time(ev1))
            finally:
                handle.set_kernel_path(rk.PATH_AUTO)
            assert handle.poll_status() == rk.RESTKV_OK
            return float(np.median(ta))

        adaptive = {"note": "restkv_evict with the adaptive window (beta 2000, B = the budget): the score kernel also "
                            "writes the per-query indicators [b, Hq, w, n] fp32, from which %d rows of top-B are taken"
                            % (case.batch * case.n_q_heads * case.w),
                    "evict_ms": time_adaptive(rk.PATH_AUTO, 5), "evict_ms_simt_kernels": time_adaptive(rk.PATH_SIMT, 2),
                    "raw_indicator_bytes": 4 * case.batch * case.n_q_heads * case.w * case.n}
        del ws_a

    # ---- eviction again during decoding (Appendix B): the compacted cache plus M generated tokens, the last w of
    #      them as the window (their own rows are the trailing, causally masked block) ----
    reevict = None
    if rank == 0 and world == 1 and not args.no_extras and case.causal_tail == 0 and case.n > case.budget + 128:
        M, w, d, G = 128, case.w, case.head_dim, case.group
        rows = case.budget + M
        case_r = case.with_(n=rows - w, causal_tail=w)
        shape_r = rk.make_shape(case_r.batch, case_r.n_q_heads, case_r.n_kv_heads, d, case_r.n_kv, w, w,
                                rk.BF16 if case.dtype == "bf16" else rk.F32)
        Kr, Vr = K[:, :, :rows].contiguous(), V[:, :, :rows].contiguous()
        scale = 1.0 / float(np.sqrt(d))
        O_r = torch.empty(case.batch, case.n_q_heads, w, d, dtype=torch.float32, device="cuda")
        L_r = torch.empty(case.batch, case.n_q_heads, w, dtype=torch.float32, device="cuda")
        ii = torch.arange(w, device="cuda").repeat(G)[:, None]
        jj = torch.arange(rows, device="cuda")[None, :] - (rows - w)
        for bi in range(case.batch):          # what the decode calls would have left behind (not timed)
            for h in range(case.n_kv_heads):
                qf = Q[bi, h * G:(h + 1) * G].float().reshape(G * w, d)
                sc = (scale * (qf @ Kr[bi, h].float().T)).masked_fill(jj > ii, float("-inf"))
                lse = torch.logsumexp(sc, dim=-1)
                O_r[bi, h * G:(h + 1) * G] = (torch.exp(sc - lse[:, None]) @ Vr[bi, h].float()).view(G, w, d)
                L_r[bi, h * G:(h + 1) * G] = lse.view(G, w)
        ws_r = torch.empty(handle.workspace_bytes(shape_r, case.budget), dtype=torch.uint8, device="cuda")

        def time_reevict(fn):
            tr = []
            for it in range(23):
                flush.zero_()
                ev0.record()
                fn()
                ev1.record()
                torch.cuda.synchronize()
                if it >= 3:
                    tr.append(ev0.elapsed_time(ev1))
            assert handle.poll_status() == rk.RESTKV_OK
            return float(np.median(tr))

        ms_a = time_reevict(lambda: handle.evict(shape_r, Q, Kr, Vr, case.ema_decay, pool, case.budget, indices, K_out,
                                                 V_out, ws_r))
        ms_b = time_reevict(lambda: handle.evict_from_lse(shape_r, Q, Kr, Vr, O_r, L_r, case.ema_decay, pool,
                                                          case.budget, indices, K_out, V_out, ws_r))
        reevict = {"note": "one re-eviction of a cache of budget + %d rows back to the budget, window = the last %d "
                           "generated tokens (causal_tail = w)" % (M, w),
                   "rows": rows, "evict_us": ms_a * 1e3, "evict_from_decode_statistics_us": ms_b * 1e3}
        del Kr, Vr, O_r, L_r, ws_r

    # ---- the output projection inside Eq. 7's norm (Eq. 4): || (o - v) W_O ||, W_O random [Hq * d, 4096] ----
    projection = None
    if rank == 0 and world == 1 and not args.no_extras and case.dtype == "bf16":
        d_model = 4096
        Wp = (torch.randn(case.n_q_heads * case.head_dim, d_model, device="cuda", generator=torch.Generator("cuda").manual_seed(7))
              / float(np.sqrt(d_model))).to(torch.bfloat16)
        factor = torch.empty(handle.output_projection_bytes(case.n_q_heads, case.head_dim), dtype=torch.uint8, device="cuda")
        ev0.record()
        handle.prepare_output_projection(case.n_q_heads, case.head_dim, d_model, rk.BF16, Wp, factor)
        ev1.record()
        torch.cuda.synchronize()
        prep_ms = ev0.elapsed_time(ev1)
        handle.set_output_projection(factor, case.n_q_heads, case.head_dim)
        try:
            tp = []
            for it in range(13):
                flush.zero_()
                ev0.record()
                step()
                ev1.record()
                torch.cuda.synchronize()
                if it >= 3:
                    tp.append(ev0.elapsed_time(ev1))
            pk = kernel_pass({"value_forms": rk.KERNEL_PASS1, "score_pool_select_compact": rk.KERNEL_PASS2}, 5)
        finally:
            handle.set_output_projection(None)
        assert handle.poll_status() == rk.RESTKV_OK
        projection = {"note": "restkv_evict with restkv_set_output_projection: the tokens' own quadratic forms v^T M v "
                              "come from a tensor-core kernel of their own (one more read of V), the rest is the same launch",
                      "d_model": d_model, "prepare_ms_once_per_layer": prep_ms, "evict_ms": float(np.median(tp)),
                      "kernels_ms": pk}
        del Wp, factor

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        hQ, hK, hV = (torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in (q_np, k_np, v_np))
        h_idx = torch.empty(BH + (keep,), dtype=torch.int32).pin_memory()
        h_Ko = torch.empty(BH + (keep, case.head_dim), dtype=torch.int16 if case.dtype == "bf16" else torch.float32)
        h_Ko = h_Ko.pin_memory()
        h_Vo = torch.empty_like(h_Ko).pin_memory()
        e2e_steps = max(2, min(args.steps, 5))

        def e2e_step():
            handle.evict_host(shape, hQ, hK, hV, case.ema_decay, pool, case.budget, h_idx, h_Ko, h_Vo, Q, K, V,
                              indices, K_out, V_out, ws)
        e2e_step()
        barrier()
        # what came back through the host buffers must be what the device path produced (not timed)
        step()
        torch.cuda.synchronize()
        e2e_ok = bool(torch.equal(h_idx, indices.cpu()) and
                      torch.equal(h_Ko.view(torch.int16) if case.dtype == "bf16" else h_Ko,
                                  (K_out.view(torch.int16) if case.dtype == "bf16" else K_out).cpu()) and
                      torch.equal(h_Vo.view(torch.int16) if case.dtype == "bf16" else h_Vo,
                                  (V_out.view(torch.int16) if case.dtype == "bf16" else V_out).cpu()))
        if not e2e_ok:
            raise SystemExit("bench.py: the host-buffer path returned other results than the device path")
        ms = 0.0
        for _ in range(e2e_steps):
            ev0.record()
            e2e_step()
            ev1.record()
            torch.cuda.synchronize()
            ms += ev0.elapsed_time(ev1)
        barrier()
        ms = max_over_ranks(ms, world, "cuda")
        h2d = sum(x.numel() * x.element_size() for x in (hQ, hK, hV))
        d2h = sum(x.numel() * x.element_size() for x in (h_idx, h_Ko, h_Vo))
        e2e = {"value": tokens_per_step * e2e_steps / (ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "outputs_equal_device_path": e2e_ok}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    kv_bytes, out_bytes = algorithmic_bytes(case, keep)
    flops = algorithmic_flops(case)
    dominant = "score_pool_select_compact" if fused else "score"
    # algorithmic bytes of the dominant kernel: K and V once plus 4 B of score per token and head, and, when it also
    # selects and gathers, the indices and the compacted cache written
    dom_bytes = kv_bytes + 4 * case.batch * case.n_kv_heads * case.n_kv
    if fused:
        dom_bytes += out_bytes + 4 * case.batch * case.n_kv_heads * keep
    achieved = dom_bytes / (kmean[dominant] * 1e-3) / 1e9
    roofline = {"bound": "hbm",
                "kernel": "tc_fused_kernel (pass 1 + merge + pass 2%s)" % (" + pooling + selection + gather" if fused else ""),
                "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                "traffic": measured_traffic(args.workload) if args.path == 0 else None,
                "peak_source": peaks["source"], "algorithmic_bytes_per_launch": dom_bytes,
                "ms_per_launch": kmean[dominant]}
    t_roof_ms = max((kv_bytes + out_bytes) / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)) * 1e3
    path_roofline = {"t_roof_ms": t_roof_ms, "ms_per_step": ms_per_step / 1.0, "frac": t_roof_ms / ms_per_step,
                     "bytes": kv_bytes + out_bytes, "flops": flops, "peak_source": peaks["source"],
                     "note": "fused path against max(bytes/HBM peak, flops/bf16 peak); K,V read once + compacted write"}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": case.dtype, "data": "synthetic",
        "config": workload_config(case, l2="flushed between steps (256 MiB write); inputs 537 MB > 126 MB L2"),
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "path_roofline": path_roofline, "kernels_ms": kmean,
        "kernels_ms_selection_as_own_kernel": kmean_split, "decode": decode, "from_lse": from_lse,
        "variants": variants, "adaptive_window": adaptive, "reevict": reevict, "output_projection": projection,
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(inp, case.budget)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
