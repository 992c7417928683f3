"""Benchmark of the SCD hot path: generated tokens/s and accepted tokens per forward on one B200.

A "step" is one SCD iteration (window forward + fused verify-and-redraft) of one decode batch.
Default arm: the CUDA library through its C ABI. `--impl reference`: the CPU oracle as it stands,
timed on the host cores, on a bounded sample of the same workload.

Prints ONE JSON line (rank 0). Under torchrun every rank decodes its own replica of the workload
(independent sequences, no data-path collective): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "generated_tokens_per_s"
UNIT = "tokens/s"

# Typed-in constants (NOT measured by a run of this file; each is labelled as such in the JSON line).
# DRAM traffic of gemm_ws_kernel relative to its algorithmic (weight) bytes, from the ncu capture
# summarised in profiles/gemm_ws_kernel_session_layer.md (dram__bytes_read.sum + dram__bytes_write.sum of
# the four GEMMs of a layer over their weight bytes: 419.9 MB for 404.75 MB). Traffic grows in proportion
# to the weight bytes (every weight is read once), so the ratio is applied to the average launch.
# None = the kernel changed since the capture.
GEMM_TRAFFIC_RATIO = 1.037
GEMM_TRAFFIC_SOURCE = "profiles/gemm_ws_kernel_session_layer.md (ncu capture; typed in, not measured by this run)"

# Tokens committed per forward on each workload, as measured by earlier runs of the CUDA arm (the oracle
# commits the same tokens: parity). Used only by the reference arm, which cannot afford whole generations,
# to convert the oracle's seconds per iteration into tokens/s.
MEASURED_ACCEPT = {"tiny": 1.6, "llamagen_xl": 5.3, "lumina_7b": 1.05, "video_4b": 1.02, "janus_like": 1.05,
                   "video_4b_top_p": 1.02}


# ------------------------------------------------------------------------------------------ helpers
def measured_peaks():
    """HBM GB/s and bf16 TFLOP/s measured on this machine (generated file), else the fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, pw, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
                except ValueError:
                    continue
                for n, v in zip(names, parts[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "power_w_max": float(max(pw)),
                "samples": len(sm), "reasons": sorted(reasons)}


def config_of(args, shape):
    """The workload description both arms print."""
    S = 2 if shape["cfg_lambda"] != 0.0 else 1
    return {"workload": args.workload, "batch": args.batch, "streams": S, "window_L": shape["window_L"],
            "prompt_len": shape["prompt_len"], "n_gen": shape["n_gen"], "top_k": shape["top_k"],
            "cfg_lambda": shape["cfg_lambda"], "coupling": args.coupling,
            "autotune": bool(getattr(args, "autotune", False)),
            "layers": shape["n_layers"],
            "truncated_for_profiling": bool(getattr(args, "layers", 0)),
            "l2": "inputs larger than L2 (weights streamed once per step)",
            "replicas": "one independent decode batch per GPU"}


def aggregate_over_ranks(elapsed, count, world, device):
    """The multi-rank reduction of a timed region: the slowest rank's time and the units of all
    ranks (replicas: no other collective touches the data path). `device` is where the two
    scalars live for the collective ("cuda" under NCCL, "cpu" under gloo)."""
    if world <= 1:
        return float(elapsed), float(count)
    import torch
    import torch.distributed as dist
    t = torch.tensor([elapsed], dtype=torch.float64, device=device)
    k = torch.tensor([float(count)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(k, op=dist.ReduceOp.SUM)
    return float(t.item()), float(k.item())


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def weight_bytes(shape) -> dict:
    """Algorithmic bytes of one iteration's weight stream (model dtype), by GEMM class."""
    es = 4 if shape["dtype"] == "f32" else 2
    d, dq = shape["d_model"], shape["n_heads"] * shape["head_dim"]
    dkv, F = shape["n_kv_heads"] * shape["head_dim"], shape["d_ffn"]
    nl = shape["n_layers"]
    # only the LM-head rows of ids that can be sampled are algorithmically needed
    lm_rows = shape["allowed_hi"] - shape["allowed_lo"] + (1 if shape["row_period"] > 0 else 0)
    return dict(gemm_qkv=nl * (dq + 2 * dkv) * d * es, gemm_o=nl * d * dq * es,
                gemm_gate_up=nl * 2 * F * d * es, gemm_down=nl * d * F * es,
                gemm_lm_head=lm_rows * d * es)


def kv_bytes_per_token(shape) -> int:
    es = 4 if shape["dtype"] == "f32" else 2
    return 2 * shape["n_layers"] * shape["n_kv_heads"] * shape["head_dim"] * es


def verify_bytes(shape, B, S, L) -> int:
    """Logit rows the fused verify pass must move: read S target rows and the draft row,
    write the post-processed row, over the ids that can be sampled."""
    V = shape["allowed_hi"] - shape["allowed_lo"]
    return B * L * V * 4 * (S + 2)


# ------------------------------------------------------------------------------------------ CPU oracle arm
def oracle_sample(shape, weights_np, cond, uncond, n_layers_sample):
    """One SCD iteration of the oracle on a model truncated to n_layers_sample layers: the window
    forward of every stream, the post-processing of every row and the vectorised verify.
    Returns the seconds it took on the host cores (the prompt's prefill is not timed)."""
    import oracle
    L, P, V = shape["window_L"], shape["prompt_len"], shape["vocab_out"]
    S = 2 if shape["cfg_lambda"] != 0.0 else 1
    sub = dict(shape, n_layers=n_layers_sample, max_seq=P + L + 8)
    om = oracle.Model(sub, weights_np, n_streams=S)
    lo, hi, seed = shape["allowed_lo"], shape["allowed_hi"], shape["seed"]
    prompts = [cond, uncond]
    if P > 1:
        for s in range(S):
            om.forward(prompts[s][:P - 1], 0, stream=s)
    drafts = np.array([oracle.fresh_draft(seed, 0, P + k, 0, lo, hi) for k in range(L)], dtype=np.int32)
    t0 = time.perf_counter()
    logits = []
    for s in range(S):
        ids = np.concatenate([prompts[s][P - 1:P], drafts[:L - 1]]).astype(np.int32)
        logits.append(om.forward(ids, P - 1, stream=s))
    Wp = np.zeros((L, V), dtype=np.uint32)
    Wq = np.zeros((L, V), dtype=np.uint32)
    Zp = np.zeros(L, dtype=np.uint64)
    Zq = np.zeros(L, dtype=np.uint64)
    for k in range(L):
        Wp[k], Zp[k] = oracle.postprocess(logits[0][k], logits[1][k] if S == 2 else None, lo, hi,
                                          shape["temperature"], shape["top_k"], shape["cfg_lambda"])
        if shape.get("top_p", 0.0):
            Wp[k], Zp[k] = oracle.top_p_filter(Wp[k], Zp[k], shape["top_p"])
        Wq[k], Zq[k] = oracle.uniform_weights(V, lo, hi)
    oracle.verify_window(Wp, Zp, Wq, Zq, drafts, P, 0, seed)
    return time.perf_counter() - t0


def run_reference(args, shape):
    """The oracle, as it stands, on the host cores: each step is one SCD iteration of the
    workload's shape on a depth-truncated copy of the model (a bounded sample), scaled to the
    full depth."""
    import torch
    import oracle
    from paper_2510_24211_b200 import synth
    rank, world, _ = dist_env()
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    nl_s = min(shape["n_layers"], args.ref_layers)
    sub = dict(shape, n_layers=nl_s)
    w = synth.make_weights(sub, seed=1234)
    wn = synth.weights_to_numpy(w)
    cond, uncond = synth.make_prompt(shape)
    S = 2 if shape["cfg_lambda"] != 0.0 else 1
    times = []
    for i in range(args.warmup_ref + args.steps_ref):
        t = oracle_sample(shape, wn, cond[0], uncond[0], nl_s)
        if i >= args.warmup_ref:
            times.append(t)
    # an iteration's cost is linear in depth apart from the LM head and the verify pass, which the
    # truncated model already carries in full; scale conservatively (all of it) by depth
    t_iter = float(np.mean(times)) * shape["n_layers"] / nl_s
    mean_a = args.assumed_accept if args.assumed_accept > 0 else MEASURED_ACCEPT.get(args.workload, 1.0)
    accept_source = "--assumed-accept" if args.assumed_accept > 0 else "typed in from earlier runs of the CUDA arm"
    value = mean_a / t_iter
    sample = (f"one SCD iteration (S={S} x L={shape['window_L']} rows) of the {args.workload} shape on the first "
              f"{nl_s} of {shape['n_layers']} layers + full LM head + verify; time scaled by depth; tokens per "
              f"forward {mean_a:.2f} ({accept_source})")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps_ref, "warmup": args.warmup_ref, "ms_per_step": t_iter * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64 accumulate over bf16 weights",
            "data": "synthetic", "config": config_of(args, shape),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ CUDA arm
def context_prompts(shape, cond, uncond, extra, seed=4321):
    """The workload's prompt followed by `extra` synthetic generated-range ids (the same in both streams, as
    generated tokens are): a stand-in for a generation that is `extra` tokens along, reached without
    generating them. Forced end-of-row positions keep their id."""
    if extra <= 0:
        return cond, uncond
    rng = np.random.default_rng(seed)
    B = cond.shape[0]
    gen = rng.integers(shape["allowed_lo"], shape["allowed_hi"], size=(B, extra)).astype(np.int32)
    if shape["row_period"] > 0:
        g = np.arange(extra)
        gen[:, g % shape["row_period"] == shape["row_period"] - 1] = shape["eol_id"]
    return np.concatenate([cond, gen], axis=1), np.concatenate([uncond, gen], axis=1)


def run_scd(args, shape):
    import torch
    from paper_2510_24211_b200 import binding as scd
    from paper_2510_24211_b200 import synth

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    scd.lib()                                            # fails loudly if libscd.so is missing

    B = args.batch
    S = 2 if shape["cfg_lambda"] != 0.0 else 1
    L = args.window if args.window > 0 else shape["window_L"]
    shape = dict(shape, window_L=L)
    P, N = shape["prompt_len"], shape["n_gen"]
    max_seq = P + N + L
    w = synth.make_weights(shape, seed=1234, device="cuda")
    model = scd.Model(shape, w, max_seq=max_seq)
    if args.gemm_splits or args.gemm_stages:
        model.scd_model_gemm_tune(args.gemm_splits, args.gemm_stages)
    cond, uncond = synth.make_prompt(shape, batch=B)

    def cfg_of(mode):
        return scd.decode_config(mode=mode, batch=B, window_L=L, temperature=shape["temperature"],
                                 top_k=shape["top_k"], cfg_lambda=shape["cfg_lambda"], seed=shape["seed"] + rank,
                                 allowed_lo=shape["allowed_lo"], allowed_hi=shape["allowed_hi"],
                                 row_period=shape["row_period"], eol_id=shape["eol_id"], alpha=args.alpha,
                                 top_p=shape.get("top_p", 0.0))

    coupling = {"scd_mc": scd.SCD_MODE_SCD_MC, "scd_gs": scd.SCD_MODE_SCD_GS, "sjd": scd.SCD_MODE_SJD,
                "alpha": scd.SCD_MODE_ALPHA}[args.coupling]
    sess = scd.Session(model, cfg_of(coupling))
    if args.att_min_ctx is not None:
        sess.scd_session_attention_min_ctx(args.att_min_ctx)
    tuned = None
    stream = torch.cuda.current_stream()
    peaks = measured_peaks()
    wb = weight_bytes(shape)
    gemm_classes = ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down", "gemm_lm_head")
    gemm_bytes = sum(wb[c] for c in gemm_classes)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def prefill_at(extra):
        """A generation `extra` tokens along: the remaining N - extra tokens are still to come."""
        c, u = context_prompts(shape, cond, uncond, extra)
        sess.scd_prefill(np.concatenate([c, u]) if S == 2 else c, n_new=N - extra)
        return P + extra

    def timed_steps(steps, extra):
        """Exactly `steps` iterations (CUDA events on the launching stream), in segments that never run past
        the end of a generation; a generation that ends is restarted (untimed) at the same context."""
        n_total = P + N
        done, tokens, total_ms, ctx_sum = 0, 0, 0.0, 0.0
        _, n_now, _ = sess.scd_step_result()
        while done < steps:
            remaining = int((n_total - n_now).max())
            if remaining <= 0:
                prefill_at(extra)                            # untimed: a new generation starts
                _, n_now, _ = sess.scd_step_result()
                continue
            seg = min(steps - done, (remaining + L - 1) // L)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(seg):
                sess.scd_step()
            e1.record(stream)
            e1.synchronize()
            total_ms += e0.elapsed_time(e1)
            _, n_after, _ = sess.scd_step_result()
            tokens += int((n_after - n_now).sum())
            ctx_sum += seg * float(n_now.mean() + n_after.mean()) / 2.0
            n_now = n_after
            done += seg
        return total_ms, tokens, ctx_sum / max(done, 1)

    def step_bytes_at(mean_ctx):
        # whole iteration: weights + KV read at the mean context of the timed region + verify rows
        return gemm_bytes + mean_ctx * S * B * kv_bytes_per_token(shape) + verify_bytes(shape, B, S, L)

    # ---- warm-up: a fresh generation, W steps -----------------------------------------------------
    start_extra = {"start": 0, "mid": N // 2, "end": max(0, N - 2 * L)}[args.context]
    prefill_at(start_extra)
    if args.autotune:
        tuned = [int(x) for x in sess.scd_autotune()]
    for _ in range(max(args.warmup, 3)):
        sess.scd_step()
    torch.cuda.synchronize()

    # ---- timed: exactly K steps ------------------------------------------------------------------
    sampler = ClockSampler(local)
    launches0 = scd.scd_kernel_launches()
    barrier()
    sampler.start()
    total_ms, tokens, mean_ctx = timed_steps(args.steps, start_extra)
    barrier()
    clocks = sampler.stop()
    launches = scd.scd_kernel_launches() - launches0

    total_ms_all, tokens_all = aggregate_over_ranks(total_ms, tokens, world, "cuda")
    value = tokens_all / (total_ms_all * 1e-3)
    ms_per_step = total_ms_all / args.steps
    accepted_per_forward = tokens / (args.steps * B)

    # ---- the same iteration at the start, the middle and the end of the context --------------------
    by_context = {}
    if world == 1 and not args.no_contexts:
        for name, extra in (("start", 0), ("mid", N // 2), ("end", max(0, N - 2 * L))):
            prefill_at(extra)
            for _ in range(3):
                sess.scd_step()
            torch.cuda.synchronize()
            ms, _, ctx = timed_steps(args.context_steps, extra)
            msps = ms / args.context_steps
            by_context[name] = {"context_tokens": ctx, "ms_per_step": msps, "bytes_per_step": step_bytes_at(ctx),
                                "step_roofline_frac": step_bytes_at(ctx) / (msps * 1e-3) / 1e9 / peaks["hbm_gbs"]}

    # ---- per-kernel attribution of an iteration (device events in front of every kernel) ----------
    prof_ms = np.zeros(len(scd.PROF_CLASSES), dtype=np.float32)
    prof_n = np.zeros(len(scd.PROF_CLASSES), dtype=np.int32)
    prefill_at(start_extra)
    for _ in range(3):
        sess.scd_step()
    n_prof = 0
    for _ in range(args.profile_steps):
        sess.scd_step_profile(prof_ms, prof_n)
        n_prof += 1
    # the same, from device time stamps inside the kernels: no events between them, so they overlap
    # (programmatic dependent launch) exactly as in the timed region
    tl_ms = np.zeros(len(scd.PROF_CLASSES), dtype=np.float32)
    tl_n = np.zeros(len(scd.PROF_CLASSES), dtype=np.int32)
    for _ in range(args.profile_steps):
        sess.scd_step_timeline(tl_ms, tl_n)
    by_class = {c: float(prof_ms[i]) / max(n_prof, 1) for i, c in enumerate(scd.PROF_CLASSES)}
    launches_by_class = {c: int(prof_n[i]) // max(n_prof, 1) for i, c in enumerate(scd.PROF_CLASSES)}
    gemm_ms_events = sum(by_class[c] for c in gemm_classes)
    gemm_launches = sum(launches_by_class[c] for c in gemm_classes)
    timeline = {c: float(tl_ms[i]) / max(n_prof, 1) for i, c in enumerate(scd.PROF_CLASSES)}
    gemm_ms_inflight = sum(timeline[c] for c in gemm_classes)
    roofline = None
    if gemm_launches > 0 and gemm_ms_events > 0:
        # headline: every launch timed on its own by CUDA events (the conservative figure: events between
        # the kernels switch their programmatic overlap off); second: the kernels as they overlap in a step
        achieved = gemm_bytes / (gemm_ms_events * 1e-3) / 1e9
        inflight = gemm_bytes / (gemm_ms_inflight * 1e-3) / 1e9 if gemm_ms_inflight > 0 else None
        roofline = {"bound": "hbm", "kernel": "gemm_ws_kernel (all weight GEMMs of an iteration)",
                    "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                    "timing": "CUDA events on the launching stream around every launch (no overlap between kernels)",
                    "bytes_per_launch": gemm_bytes / gemm_launches,
                    "us_per_launch": gemm_ms_events * 1e3 / gemm_launches, "launches_per_step": gemm_launches,
                    "achieved_inflight": inflight,
                    "frac_inflight": inflight / peaks["hbm_gbs"] if inflight else None,
                    "us_per_launch_inflight": gemm_ms_inflight * 1e3 / gemm_launches,
                    "inflight_note": "device time stamps inside the kernels, completion to completion, kernels "
                                     "overlapping (programmatic dependent launch) as in the timed region",
                    "traffic": (gemm_bytes / gemm_launches) * GEMM_TRAFFIC_RATIO if GEMM_TRAFFIC_RATIO else None,
                    "traffic_source": GEMM_TRAFFIC_SOURCE}
    step_bytes = step_bytes_at(mean_ctx)
    step_roofline = {"bound": "hbm", "achieved": step_bytes / (ms_per_step * 1e-3) / 1e9 if world == 1 else None,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "bytes_per_step": step_bytes,
                     "mean_context_tokens": mean_ctx}
    if step_roofline["achieved"]:
        step_roofline["frac"] = step_roofline["achieved"] / peaks["hbm_gbs"]
    # the fused verify kernel: by bytes it belongs to the HBM roofline, in practice it is bound by the
    # latency of its chain of row-wide exchanges (see profiles/); reported so that the gap is visible
    verify_roofline = None
    if by_class.get("verify", 0.0) > 0:
        vb = verify_bytes(shape, B, S, L)
        vach = vb / (by_class["verify"] * 1e-3) / 1e9
        verify_roofline = {"bound": "hbm", "kernel": "verify kernel", "achieved": vach, "peak": peaks["hbm_gbs"],
                           "unit": "GB/s", "frac": vach / peaks["hbm_gbs"], "bytes_per_launch": vb,
                           "us_per_launch": by_class["verify"] * 1e3,
                           "timing": "CUDA events around the launch (includes the launch gap)"}

    # ---- the same library's vanilla AR path (speed-up denominator) --------------------------------
    ar_ms, ar_tokens_per_s = None, None
    if not args.no_ar:
        ar = scd.Session(model, cfg_of(scd.SCD_MODE_AR))
        c, u = context_prompts(shape, cond, uncond, start_extra)
        ar.scd_prefill(np.concatenate([c, u]) if S == 2 else c, n_new=N - start_extra)
        for _ in range(3):
            ar.scd_step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.ar_steps):
            ar.scd_step()
        e1.record(stream)
        e1.synchronize()
        ar_ms = e0.elapsed_time(e1) / args.ar_steps
        ar_tokens_per_s = B / (ar_ms * 1e-3)
        ar.close()

    # ---- prefill of the workload's prompt (compute-bound for long prompts) ------------------------
    prefill = None
    if world == 1:
        prompts0 = np.concatenate([cond, uncond]) if S == 2 else cond
        sess.scd_prefill(prompts0, n_new=N)              # warm (tensor maps, kernels)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        sess.scd_prefill(prompts0, n_new=N)
        torch.cuda.synchronize()
        pf_s = time.perf_counter() - t0
        params = sum(wb[c] for c in ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down")) / (4 if shape["dtype"] == "f32" else 2)
        flops = 2.0 * params * S * B * max(P - 1, 0)
        prefill = {"prompt_tokens": P, "streams": S * B, "ms": pf_s * 1e3, "timing": "wall clock around scd_prefill (host copy in, synchronised)",
                   "tflops": flops / pf_s / 1e12 if pf_s > 0 else None,
                   "frac_of_bf16_sustained": flops / pf_s / 1e12 / peaks["bf16_tflops_sustained"] if pf_s > 0 else None,
                   "flops_note": "2 x layer parameters x prompt rows (attention and the second activation plane not counted)"}

    # ---- end to end through the public calls: host prompt in, host tokens out ---------------------
    e2e = None
    if not args.no_e2e:
        prompts = np.concatenate([cond, uncond]) if S == 2 else cond
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        sess.scd_prefill(prompts, n_new=N)
        toks, st = sess.scd_generate()
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        e2e_tokens = B * N
        e2e_s_all, e2e_tokens_all = aggregate_over_ranks(e2e_s, e2e_tokens, world, "cuda")
        e2e_value = e2e_tokens_all / e2e_s_all
        fw = max(int(st.forwards), 1)
        e2e = {"value": e2e_value, "unit": UNIT,
               "what": "scd_prefill(host prompt) + scd_generate(host tokens out), wall clock, whole generation",
               "forwards": int(st.forwards), "accepted_per_forward": N / fw, "seconds": e2e_s,
               "ms_per_forward": e2e_s * 1e3 / fw,
               "h2d_bytes_per_step": prompts.nbytes / fw, "d2h_bytes_per_step": toks.nbytes / fw}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if shape["dtype"] == "bf16" else "f32",
            "data": "synthetic",
            "config": dict(config_of(args, shape), context=args.context),
            "accepted_tokens_per_forward": accepted_per_forward,
            "speedup_vs_own_ar": (value / world / ar_tokens_per_s) if ar_tokens_per_s else None,
            "ar_tokens_per_s": ar_tokens_per_s,
            "ar_ms_per_step": ar_ms,
            "scd_step_over_ar_step": (ms_per_step / ar_ms) if ar_ms else None,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "step_roofline": step_roofline, "verify_roofline": verify_roofline,
            "by_context": by_context, "prefill": prefill,
            "autotuned_k_splits": tuned,
            "ms_by_kernel_class": {c: round(v, 5) for c, v in by_class.items() if v > 0},
            "ms_by_kernel_class_overlapped": {c: round(v, 5) for c, v in timeline.items() if v > 0}}

    # ---- the CPU oracle on the host cores, rank 0 at N = 1 only -----------------------------------
    if world == 1 and not args.no_cpu_baseline:
        cores = os.cpu_count() or 1
        nl_s = min(shape["n_layers"], args.ref_layers)
        keep = ("tok_emb", "final_norm", "lm_head")
        wn = {k: synth.to_numpy(w[k]) for k in keep}
        for k in synth.LAYER_KEYS:
            wn[k] = [synth.to_numpy(t) for t in w[k][:nl_s]]
        t_s = oracle_sample(shape, wn, cond[0], uncond[0], nl_s)
        t_iter = t_s * shape["n_layers"] / nl_s
        line["cpu_baseline"] = {
            "value": accepted_per_forward / t_iter, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": (f"one SCD iteration (S={S} x L={L} rows) on the first {nl_s} of {shape['n_layers']} layers "
                       f"+ full LM head + verify, {t_s:.1f} s; scaled by depth to {t_iter:.1f} s per iteration; "
                       f"tokens per forward taken from the GPU run")}
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=600)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="scd", choices=["scd", "reference"])
    ap.add_argument("--workload", default="lumina_7b")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--profile-steps", type=int, default=10)
    ap.add_argument("--ar-steps", type=int, default=100)
    ap.add_argument("--ref-layers", type=int, default=12, help="depth of the oracle's timed sample")
    ap.add_argument("--assumed-accept", type=float, default=0.0,
                    help="tokens per forward used to convert the oracle's iteration time (reference arm)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gemm-splits", type=int, default=0, help="tuning: force the K slices of every GEMM (0 = automatic)")
    ap.add_argument("--coupling", choices=("scd_mc", "scd_gs", "sjd", "alpha"), default="scd_mc",
                    help="redraft rule: maximal coupling (Algorithm 6, the metric's), Gumbel sharing "
                         "(Algorithm 7), independent (SJD, Algorithm 2), alpha-coupling (Algorithm 5)")
    ap.add_argument("--alpha", type=float, default=0.5, help="--coupling alpha: probability of the coupled redraft")
    ap.add_argument("--autotune", action="store_true",
                    help="let the library pick the K slicing of the layer GEMMs by timing window forwards "
                         "(changes the order of fp32 additions, hence possibly the sampled tokens)")
    ap.add_argument("--gemm-stages", type=int, default=0, help="tuning: force the ring depth of every GEMM (0 = automatic)")
    ap.add_argument("--no-ar", action="store_true", help="skip the vanilla-AR arm (short profiling runs)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end arm (short profiling runs)")
    ap.add_argument("--context", choices=("start", "mid", "end"), default="start",
                    help="where in the generation the timed region starts (a synthetic prompt of that length is prefilled)")
    ap.add_argument("--no-contexts", action="store_true", help="skip the start / mid / end measurements")
    ap.add_argument("--context-steps", type=int, default=24, help="iterations timed at each of start / mid / end")
    ap.add_argument("--window", type=int, default=0, help="Jacobi window L (0 = the workload's)")
    ap.add_argument("--att-min-ctx", type=int, default=None,
                    help="tuning: committed context from which the tcgen05 attention kernel is used (default: the library's; "
                         "0 = always, -1 = never)")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling only: truncate the decoder to this many layers (a small model for ncu captures; "
                         "the line is marked and is not a benchmark of the workload)")
    args = ap.parse_args()
    from paper_2510_24211_b200 import synth
    shape = dict(synth.WORKLOADS[args.workload])
    if args.layers > 0:
        shape["n_layers"] = min(shape["n_layers"], args.layers)
    if args.impl == "reference":
        # the oracle's steps are tens of seconds each: bound the run
        args.steps_ref = max(1, min(args.steps, 3))
        args.warmup_ref = 0 if args.warmup == 0 else 1
        run_reference(args, shape)
    else:
        run_scd(args, shape)


if __name__ == "__main__":
    main()
