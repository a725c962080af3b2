#!/usr/bin/env python
"""Benchmark of the Pacer hot path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input:
prefill of a seeded random prompt, then the draft / pre-verify / verify / accept
loop until max_new tokens exist.  The headline value is generated tokens per
second of the decode loop at batch 1, timed on the device with CUDA events
(prefill excluded, inputs resident in HBM).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

The path does not shard (one sequence is a strict chain): with --gpus N > 1 each
rank runs an independent replica and the value is the sum ("replicas only").
--impl reference times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_01274_b200 import synth  # noqa: E402

METRIC = "generated tokens/s at batch 1 (device-timed) + HBM GB/s fraction of peak in verify"
UNIT = "tokens/s"
PACER_T0 = 0.5      # threshold of the headline "Pacer" row (the only value that varies the window
                    # with an untrained pre-verification layer)


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def verify_bytes(cfg: synth.PairConfig, ctx_len: int, rows: int) -> float:
    """Algorithmic bytes of one target verify forward: weights once, live KV of every sequence once, new KV written
    (rows = verify rows per sequence)."""
    t = cfg.target
    return t.streamed_weight_bytes() + cfg.batch * t.kv_bytes_per_token() * (ctx_len + rows)


def oracle_sample(cfg: synth.PairConfig, pair_cpu, prompt, n_prompt_s, n_steps_s, t0):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: the first n_prompt_s prompt tokens
    (prefill, untimed like the GPU arm's), then n_steps_s draft-and-verify steps of Algorithm 1 (timed).
    Returns (tokens/s, tokens made, seconds)."""
    from oracle import pacer_oracle as orc
    T = orc.OracleModel(cfg.target, pair_cpu["target"], pair_cpu["succ_T"], cfg.succ_bias)
    D = orc.OracleModel(cfg.draft, pair_cpu["draft"], pair_cpu["succ_D"], cfg.succ_bias)
    B = orc.OracleModel(synth.preverify_shape(cfg.draft), pair_cpu["preverify"])
    o = orc.Pacer(T, D, B, n_prompt_s + n_steps_s * (cfg.gamma_cap + 1) + cfg.gamma_cap + 2, b=cfg.block_b,
                  gamma_cap=cfg.gamma_cap, t0=t0, rho=cfg.rho)
    o.prefill(prompt[:n_prompt_s])
    t = time.perf_counter()
    made = 0
    for _ in range(n_steps_s):
        while o.drafting:
            o.draft_block(); o.preverify()
        o.verify()
        made += o.accept() + 1
    dt = time.perf_counter() - t
    return made / dt, made, dt


def kernel_source_digest() -> str:
    """sha1 over the CUDA sources: ties the DRAM counters kept under profiles/ to the kernel they were taken on."""
    import hashlib
    h = hashlib.sha1()
    d = os.path.join(ROOT, "paper_2602_01274_b200", "csrc")
    for f in sorted(os.listdir(d)):
        if f.endswith((".cu", ".cuh")):
            h.update(open(os.path.join(d, f), "rb").read())
    return h.hexdigest()[:16]


def measured_traffic_ratio():
    """(dram bytes of a verify launch / its algorithmic bytes, note) from the ncu counters kept with the profile
    summaries, or (None, why) when there are none for the kernel as it is now."""
    p = os.path.join(ROOT, "profiles", "k_forward_dram_counters.txt")
    if not os.path.exists(p):
        return None, "no ncu counters on record"
    kv = dict(line.split(None, 1) for line in open(p) if line.strip() and not line.startswith("#"))
    if kv.get("kernel_source_digest", "").strip() != kernel_source_digest():
        return None, "the kernel has changed since the ncu counters were taken"
    return float(kv["dram_bytes_over_algorithmic_bytes"]), kv.get("capture", "").strip()


def verify_forward_numbers(ctx, cfg, prompt, n_ver, n_warm):
    """Times the target verify forward with a full draft window (gamma_cap + 1 rows).  The forward is ONE launch
    of the persistent kernel k_forward, so the dominant kernel's launch duration is the forward's: measured twice,
    with torch events around n_ver launches on the context's stream, and launch by launch with the library's own
    event pairs (pacer_profile_*)."""
    ctx.pacer_prefill(prompt, cfg.max_new, cfg.gamma_max, -1.0)
    for _ in range(cfg.gamma_cap // cfg.block_b):
        for _ in range(cfg.block_b):
            ctx.pacer_draft_step()
        ctx.pacer_preverify()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(ctx.stream)
    ctx.pacer_draft_step()             # (a no-op forward: the window is full) launch cost of an idle forward
    e1.record(ctx.stream)
    torch.cuda.synchronize()
    idle_us = e0.elapsed_time(e1) * 1e3
    for _ in range(n_warm):
        ctx.pacer_verify()            # same rows every time: the state does not advance without accept
    e0.record(ctx.stream)
    for _ in range(n_ver):
        ctx.pacer_verify()
    e1.record(ctx.stream)
    torch.cuda.synchronize()
    ver_ms = e0.elapsed_time(e1) / n_ver
    ctx.pacer_profile_begin()
    for _ in range(n_ver):
        ctx.pacer_verify()
    fwd_ms, weight_bytes, fwd_n = ctx.pacer_profile_end()
    peak, peak_kind = _peaks()
    ctx_len = cfg.n_prompt - 1
    vbytes = verify_bytes(cfg, ctx_len, cfg.gamma_cap + 1)
    launch_ms = fwd_ms / max(1, fwd_n)
    gbs = vbytes / (launch_ms * 1e-3) / 1e9
    ratio, ratio_note = measured_traffic_ratio()
    roofline = {"bound": "hbm", "kernel": "k_forward (one launch = one verify forward)", "achieved": gbs, "peak": peak,
                "unit": "GB/s", "frac": gbs / peak, "peak_kind": f"of {peak_kind}",
                "traffic": None if ratio is None else vbytes * ratio,
                "traffic_note": ratio_note if ratio is None else
                "from profiles: dram read + write bytes of one launch in the ncu capture of a layer-cut model (%s), "
                "%.3f x its algorithmic bytes, scaled to this launch by its algorithmic bytes" % (ratio_note, ratio),
                "launches_timed": fwd_n, "bytes_per_launch": vbytes, "weight_bytes_per_launch": weight_bytes / max(1, fwd_n),
                "ms_per_launch": launch_ms}
    verify = {"ms": ver_ms, "algorithmic_gb": vbytes / 1e9, "achieved_gbs": vbytes / (ver_ms * 1e-3) / 1e9,
              "frac_of_measured_peak": vbytes / (ver_ms * 1e-3) / 1e9 / peak,
              "frac_of_8tbs": vbytes / (ver_ms * 1e-3) / 1e9 / 8000.0, "rows": cfg.batch * (cfg.gamma_cap + 1), "ctx": ctx_len,
              "sequences": cfg.batch, "idle_forward_us": idle_us}
    return {"roofline": roofline, "verify_forward": verify}


def aggregate_replicas(dec_ms: float, e2e_s: float, tokens: float, steps: int, world: int, device="cpu"):
    """Whole-job numbers of `world` independent replicas (the path does not shard: no data-path collective):
    tokens summed over ranks, divided by the slowest rank's time.  Returns (tokens/s device-timed, tokens/s end to
    end, ms per step).  Only this reporting step talks between ranks (one MAX and one SUM all-reduce)."""
    if world <= 1:
        return tokens / (dec_ms * 1e-3), tokens / e2e_s, dec_ms / steps
    import torch.distributed as dist
    t = torch.tensor([dec_ms, e2e_s, float(tokens)], device=device, dtype=torch.float64)
    mx = t.clone(); dist.all_reduce(mx, op=dist.ReduceOp.MAX)
    sm = t.clone(); dist.all_reduce(sm, op=dist.ReduceOp.SUM)
    return sm[2].item() / (mx[0].item() * 1e-3), sm[2].item() / mx[1].item(), mx[0].item() / steps


def batched_sweep(args, cfg, ctx, prompts, workload, mode, seed, rank, local_rank, world, dev, barrier):
    """The batched long-context configuration: independent sequences share every forward, each with its own
    adaptive window and ragged accept / rollback.  Run as the threshold ablation {always pass = fixed window, 0.3,
    0.5, 0.7}; the headline value is the t0 = 0.5 run (all sequences' tokens over the decode time)."""
    thresholds = [("always_pass", -1.0), ("0.3", 0.3), ("0.5", 0.5), ("0.7", 0.7)]
    for _ in range(max(1, min(args.warmup, 1))):           # a full run takes seconds: one is enough to warm up
        ctx.pacer_generate(prompts, cfg.max_new, cfg.gamma_max, PACER_T0, mode, seed)
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    sweep, dec_ms, e2e_s, tok, launches = {}, 0.0, 0.0, 0, 0
    wall0 = time.perf_counter()
    for name, t0 in thresholds:
        reps = args.steps if t0 == PACER_T0 else 1
        for _ in range(reps):
            ts = time.perf_counter()
            toks, ns, dl, al, st = ctx.pacer_generate(prompts, cfg.max_new, cfg.gamma_max, t0, mode, seed)
            torch.cuda.synchronize()
            dt = time.perf_counter() - ts
            if t0 == PACER_T0:
                dec_ms += st["ms_decode"]; e2e_s += dt; tok += cfg.batch * cfg.max_new; launches += st["n_kernel_launches"]
        gam = np.concatenate([dl[q, : ns[q]] for q in range(cfg.batch)])
        acc = np.concatenate([al[q, : ns[q]] for q in range(cfg.batch)])
        sweep[name] = {"tokens_per_s": cfg.batch * cfg.max_new / (st["ms_decode"] * 1e-3), "tau": float(acc.mean()),
                       "mean_gamma": float(gam.mean()), "steps_per_sequence": [int(v) for v in ns],
                       "forwards": {"draft": st["n_draft_fwd"], "preverify": st["n_mb_calls"], "target": st["n_target_fwd"]},
                       "ms_prefill": st["ms_prefill"], "ms_decode": st["ms_decode"]}
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop()
    vf = verify_forward_numbers(ctx, cfg, prompts, 5, 2)
    value, e2e_val, ms_step = aggregate_replicas(dec_ms, e2e_s, tok, args.steps, world, dev)
    if rank != 0:
        return
    print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                      "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                      "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload, "clocks": clocks,
                      "gpu_launches": int(launches),
                      "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": int(prompts.nbytes),
                              "d2h_bytes_per_step": int(cfg.batch * (4 * cfg.max_new * 3 + 4) + 128),
                              "note": "pacer_generate with host prompts and host outputs; prefill inside the timed region"},
                      "roofline": vf["roofline"], "verify_forward": vf["verify_forward"],
                      "threshold_sweep": sweep, "wall_s_timed_region": wall}))


def pair_to_cpu(pair):
    return {k: ({n: t.cpu() for n, t in v.items()} if isinstance(v, dict) else v.cpu()) for k, v in pair.items()}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="33b_1b3",
                    help="synthetic pair (default: the largest single-GPU batch-1 configuration)")
    ap.add_argument("--impl", default="pacer", choices=["pacer", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-baselines", action="store_true",
                    help="only the timed Pacer runs and the verify-forward timing: no autoregressive / fixed-window / "
                         "optimal-window runs (the short command the ncu launch list is taken on)")
    ap.add_argument("--cpu-sample-steps", type=int, default=1,
                    help="draft-and-verify steps of Algorithm 1 the CPU oracle is timed on")
    ap.add_argument("--preverify", default="trained", choices=["trained", "random"],
                    help="trained: the pre-verification layer is trained on this box before the timed region, with the "
                         "paper's label recipe on the synthetic pair (untimed set-up, about a minute); random: N(0,0.02) weights")
    ap.add_argument("--train-prompts", type=int, default=0,
                    help="prompts the pre-verification layer is trained on (default: 1024, or 256 for targets above "
                         "10 B parameters, whose responses take longer to generate)")
    ap.add_argument("--t0", type=float, default=None,
                    help="initial threshold of the Pacer row (default: the best of {0.3, 0.5, 0.7} in an untimed pre-sweep "
                         "with a trained layer, 0.5 with a random one)")
    ap.add_argument("--sample", action="store_true", help="temperature-1 rejection sampling (Philox seed 1) instead of greedy")
    ap.add_argument("--only", default="all", choices=["all", "verify"],
                    help="verify: short prefill, one full draft window, then timed verify forwards only "
                         "(the small, few-launch command the ncu captures use)")
    ap.add_argument("--layers", type=int, default=0, help="with --only verify: keep this many target layers")
    ap.add_argument("--n-prompt", type=int, default=0, help="with --only verify: prompt length override")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = synth.CONFIGS[args.config]
    if args.only == "verify":
        import dataclasses
        tgt = dataclasses.replace(cfg.target, n_layers=args.layers) if args.layers else cfg.target
        cfg = dataclasses.replace(cfg, target=tgt, n_prompt=args.n_prompt or cfg.n_prompt)
    t0 = PACER_T0
    workload = {"workload": f"{cfg.name}: target {cfg.target.n_layers}L d={cfg.target.d_model}, draft "
                            f"{cfg.draft.n_layers}L d={cfg.draft.d_model}, prompt {cfg.n_prompt}, new {cfg.max_new}, "
                            f"gamma_max {cfg.gamma_max}, b {cfg.block_b}, rho {cfg.rho}, t0 {t0}, "
                            f"{'sampling T=1 seed 1' if args.sample else 'greedy'}, batch {cfg.batch}",
                "weights": "N(0,0.02) seed 0, planted successor bias +8, agreement %.2f" % cfg.agree,
                "l2": "inputs (%.1f GB of weights per forward) exceed L2; no flush needed" % (cfg.target.streamed_weight_bytes() / 1e9)}

    if args.impl == "reference":
        if rank != 0:
            return
        dev = "cuda:0" if torch.cuda.is_available() else "cpu"
        workload["preverify"] = "random N(0,0.02) weights (the cost of a step does not depend on them)"
        pair = pair_to_cpu(synth.make_pair(cfg, seed=0, device=dev))
        prompt = synth.make_prompts(cfg.target.vocab, 1, cfg.n_prompt, seed=0)[0].numpy()
        vals = []
        for i in range(args.warmup + args.steps):
            v, made, dt = oracle_sample(cfg, pair, prompt, 2, args.cpu_sample_steps, t0)
            if i >= args.warmup:
                vals.append((v, made, dt))
        tot_tok = sum(m for _, m, _ in vals); tot_t = sum(d for _, _, d in vals)
        val = tot_tok / tot_t
        cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count()))
        sample = (f"per step: first 2 prompt tokens prefilled (untimed), then {args.cpu_sample_steps} draft-and-verify "
                  f"step(s) of Algorithm 1 timed")
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / max(1, len(vals)),
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                          "data": "synthetic", "config": workload,
                          "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
                          "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl")
    from paper_2602_01274_b200 import binding as b

    pair = synth.make_pair(cfg, seed=0, device=dev)
    train_report = None
    if args.preverify == "trained" and args.only == "all":
        # Section 3.3: the target's responses to seeded random prompts, drafts from every prefix, labels up to the
        # first mismatch, cross-entropy, AdamW.  Plain PyTorch, outside the decoding path and outside the timed region.
        from paper_2602_01274_b200 import train_preverify
        n_train = args.train_prompts or (1024 if cfg.target.n_params() < 10e9 else 256)
        tensors, train_report = train_preverify.train(cfg, pair, dev, n_prompts=n_train, epochs=12, lr=1e-3,
                                                      batch_prompts=64 if cfg.draft.n_params() < 5e8 else 32,
                                                      log=lambda m: print(m, file=sys.stderr, flush=True))
        pair["preverify"] = {k: v.to(dev) for k, v in tensors.items()}
        torch.cuda.empty_cache()
        workload["preverify"] = ("trained on this box before the timed region: %d seeded prompts, %d epochs, held-out AUC %.3f"
                                 % (train_report["prompts"], train_report["epochs"], train_report["held_out_auc"]))
    else:
        workload["preverify"] = "random N(0,0.02) weights (carries no signal)"
    prompt = synth.make_prompts(cfg.target.vocab, cfg.batch, cfg.n_prompt, seed=rank).numpy()
    if cfg.batch == 1:
        prompt = prompt[0]
    max_ctx = cfg.n_prompt + cfg.max_new + cfg.gamma_cap + 2
    ctx = b.Context(b.make_cfg(cfg.target, cfg.draft, cfg.batch, max_ctx, cfg.gamma_cap, cfg.block_b, cfg.rho, 0,
                               cfg.succ_bias), device=dev)
    b.load_pair(ctx, pair)
    if cfg.batch > 1:
        del pair
        torch.cuda.empty_cache()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.only == "verify":
        if rank == 0:
            print(json.dumps({"only": "verify", "config": workload, **verify_forward_numbers(ctx, cfg, prompt, args.steps,
                                                                                             args.warmup)}))
        return

    mode, seed = (b.PACER_SAMPLE, 1) if args.sample else (b.PACER_GREEDY, 0)
    if cfg.batch > 1:
        return batched_sweep(args, cfg, ctx, prompt, workload, mode, seed, rank, local_rank, world, dev, barrier)
    t0_sweep = None
    if args.t0 is not None:
        t0 = args.t0
    elif train_report is not None:
        # the paper picks its threshold per task (appendix on evaluation parameters): an untimed sweep does it here
        t0_sweep = {}
        for cand in (0.3, 0.5, 0.7):
            _, _, _, _, s_ = ctx.pacer_generate(prompt, cfg.max_new, cfg.gamma_max, cand, mode, seed)
            t0_sweep[cand] = cfg.max_new / (s_["ms_decode"] * 1e-3)
        t0 = max(t0_sweep, key=t0_sweep.get)
    workload["workload"] = workload["workload"].replace("t0 %s" % PACER_T0, "t0 %s" % t0)
    for _ in range(args.warmup):
        ctx.pacer_generate(prompt, cfg.max_new, cfg.gamma_max, t0, mode, seed)
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    dec_ms, tok, launches, e2e_s = 0.0, 0, 0, 0.0
    stats_all = []
    wall0 = time.perf_counter()
    for _ in range(args.steps):
        ts = time.perf_counter()
        toks, ns, dl, al, st = ctx.pacer_generate(prompt, cfg.max_new, cfg.gamma_max, t0, mode, seed)
        torch.cuda.synchronize()
        e2e_s += time.perf_counter() - ts
        dec_ms += st["ms_decode"]; tok += cfg.max_new; launches += st["n_kernel_launches"]
        stats_all.append((st, ns[0], dl[0, : ns[0]].copy(), al[0, : ns[0]].copy()))
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop()

    if args.no_baselines:
        vf = verify_forward_numbers(ctx, cfg, prompt, 3, 1)
        value, e2e_val, ms_step = aggregate_replicas(dec_ms, e2e_s, tok, args.steps, world, dev)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                              "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                              "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload,
                              "clocks": clocks, "gpu_launches": int(launches),
                              "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": int(prompt.nbytes),
                                      "d2h_bytes_per_step": int(4 * cfg.max_new * 3 + 4 + 128)},
                              "roofline": vf["roofline"], "verify_forward": vf["verify_forward"]}))
        return

    # baselines on the same kernels (outside the timed region): autoregressive and fixed windows
    ar_tok, ar_st = ctx.pacer_generate_ar(prompt, cfg.max_new, mode, seed)
    ar_tps = cfg.max_new / (ar_st["ms_decode"] * 1e-3)
    lossless = None if args.sample else bool((ar_tok[0] == toks[0]).all())
    mismatch = None
    if lossless is False:
        # greedy outputs may part ways only where the target's two best logits tie within the tolerance: show the tie
        i = int(np.nonzero(ar_tok[0] != toks[0])[0][0])
        ctx.pacer_generate_ar(prompt, i + 1)
        lg = ctx.pacer_read_buffer(b.BUF_VERIFY_LOGITS, np.float32, cfg.target.vocab)
        top = np.argsort(lg)[-2:][::-1]
        mismatch = {"new_token_index": i, "ar_top2_logits": [float(lg[top[0]]), float(lg[top[1]])],
                    "ar_top2_margin": float(lg[top[0]] - lg[top[1]]), "tolerance": 2e-2}
    fixed, fixed_fwd, logs_cap = {}, {}, None
    for g in range(cfg.block_b, cfg.gamma_cap + 1, cfg.block_b):
        _, ns2, dl2, al2, s2 = ctx.pacer_generate(prompt, cfg.max_new, g, -1.0, mode, seed)
        fixed[g] = cfg.max_new / (s2["ms_decode"] * 1e-3)
        fixed_fwd[g] = {"draft": s2["n_draft_fwd"], "preverify": s2["n_mb_calls"], "target": s2["n_target_fwd"]}
        if g == cfg.gamma_cap:
            logs_cap = (dl2[0, : ns2[0]].copy(), al2[0, : ns2[0]].copy())
    best_g = max(fixed, key=fixed.get)

    # Realised acceptance by draft position, from the run with the largest window (the analogue of the paper's
    # acceptance-rate-versus-draft-position curve): of the steps that drafted position i, the share in which it was accepted.
    dl_cap, al_cap = logs_cap
    accept_by_pos = [float((al_cap >= i).sum() / max(1, (dl_cap >= i).sum())) for i in range(1, cfg.gamma_cap + 1)]
    # Oracle-knowledge optimum (Section 3.1): replay with every step's window set to the accepted length L_A* of
    # that step in the largest-window run (L_A* is capped by that window).
    opt = None
    if not args.sample:
        tok_o, ns_o, dl_o, al_o, s_o = ctx.pacer_generate_sched(prompt, cfg.max_new, al_cap, mode, seed)
        opt = {"tokens_per_s": cfg.max_new / (s_o["ms_decode"] * 1e-3),
               "forwards": {"draft": s_o["n_draft_fwd"], "preverify": 0, "target": s_o["n_target_fwd"]},
               "mean_window": float(al_cap.mean()), "all_drafts_accepted": bool((al_o[0, : ns_o[0]] == dl_o[0, : ns_o[0]]).all()),
               "same_tokens": bool((tok_o[0] == toks[0]).all()),
               "note": "windows = accepted lengths of the run with the largest fixed window (capped at gamma_cap)"}

    vf = verify_forward_numbers(ctx, cfg, prompt, 10, 3)
    roofline, verify = vf["roofline"], vf["verify_forward"]

    value, e2e_val, ms_step = aggregate_replicas(dec_ms, e2e_s, tok, args.steps, world, dev)
    if rank != 0:
        return

    st, ns, dl, al = stats_all[-1]
    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload,
           "clocks": clocks, "gpu_launches": int(launches),
           "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": int(prompt.nbytes),
                   "d2h_bytes_per_step": int(4 * cfg.max_new * 3 + 4 + 128),
                   "note": "pacer_generate with host prompt and host outputs; prefill inside the timed region"},
           "roofline": roofline, "verify_forward": verify,
           "loop": {"tokens_per_s_ar_same_kernels": ar_tps, "speedup_vs_ar": value / ar_tps,
                    "tokens_per_s_fixed_gamma": fixed, "best_fixed_gamma": best_g,
                    "speedup_vs_best_fixed": value / fixed[best_g], "tau": float(al.mean()),
                    "mean_gamma": float(dl.mean()), "steps": int(ns),
                    "forwards": {"pacer": {"draft": st["n_draft_fwd"], "preverify": st["n_mb_calls"], "target": st["n_target_fwd"]},
                                 "fixed_gamma": fixed_fwd, "autoregressive": {"target": ar_st["n_target_fwd"]}},
                    "accept_rate_by_draft_position": accept_by_pos,
                    "optimal_window": opt, "threshold_pre_sweep_tokens_per_s": t0_sweep,
                    "preverify_training": train_report,
                    "ms_prefill": st["ms_prefill"], "lossless_vs_gpu_ar": lossless,
                    "first_mismatch_vs_gpu_ar": mismatch},
           "wall_s_timed_region": wall}
    if not args.no_cpu_baseline:
        try:
            v, made, dt = oracle_sample(cfg, pair_to_cpu(pair), prompt, 2, args.cpu_sample_steps, t0)
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": int(os.environ.get("OMP_NUM_THREADS", os.cpu_count())),
                                   "kind": "oracle",
                                   "sample": f"first 2 prompt tokens prefilled (untimed), then {args.cpu_sample_steps} "
                                             f"draft-and-verify step(s) of Algorithm 1 ({made} tokens in {dt:.1f} s)"}
        except Exception as ex:  # the baseline must not take the GPU numbers down with it
            out["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": 0, "kind": "oracle", "sample": f"failed: {ex}"}
    print(json.dumps(out))


if __name__ == "__main__":
    main()
