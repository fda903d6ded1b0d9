#!/usr/bin/env python
"""Benchmark of the SpecDiff draft–verify–accept round on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one whole round (T drafter evaluations, one target verification, acceptance, commit)
of a batch-1 generation on the GPT-2-small-shaped bf16 pair (12L d768 target and drafter, V = 50257,
prompt 256 random ids, gamma = 16, T = 8, 256 new tokens).  When a generation reaches its 256 tokens
the next one (next prompt seed) starts on the same context (sdd_reset); set-up, the context's first
generation (which captures the round graphs) and prefill are outside the timed segments.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

WORKLOAD = "small_bf16"
METRIC = "SpecDiff generated tokens/s at bs=1"
UNIT = "tokens/s"
CONFIG = {"workload": "bf16 12L d768 target + 12L d768 masked-diffusion drafter, V=50257, prompt 256, "
                      "gamma=16, T=8, batch 1, 256 new tokens",
          "l2": "no flush: consecutive rounds of one generation; each round streams ~0.5 GB of weights (> 126 MB L2)",
          "graphs": "one context serves all generations (sdd_reset); its first, untimed generation captures the round graphs",
          "multi_gpu": "independent replicas, no collective on the data path"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "tf_burst": d["bf16_tflops"], "tf_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100", "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        for r in rows:
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.strip().lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(np.max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


# ----------------------------------------------------------------------------------------------
# algorithmic work per kernel category of one round (batch 1): (amount, unit-kind)
# ----------------------------------------------------------------------------------------------
def round_work(wl, c: int):
    q, p = wl.drafter, wl.target
    G, T, V = wl.gamma, wl.T, p.vocab
    L = c + G
    w = {}
    w["gemm_drafter"] = (T * 2.0 * L * 12 * q.d_model ** 2 * q.n_layer, "flop")
    w["head_drafter"] = (T * 2.0 * G * q.d_model * V, "flop")
    w["attn_drafter"] = (T * 4.0 * L * L * q.d_model * q.n_layer, "flop")
    w["gemm_target"] = (12.0 * p.d_model ** 2 * p.n_layer * 2, "byte")              # weights streamed once
    w["head_target"] = (V * p.d_model * 2.0 + (G + 1) * V * 4.0, "byte")
    w["attn_target"] = (2.0 * p.n_layer * c * p.d_model * 2, "byte")                # K and V of the cache
    w["row_stats"] = ((G + 1) * V * 4.0, "byte")
    w["accept"] = (5.0 * V * 4, "byte")
    w["sample"] = (2.0 * G * V * 4, "byte")
    w["layernorm"] = (T * (2 * q.n_layer) * L * q.d_model * 6.0 + 2 * p.n_layer * (G + 1) * p.d_model * 6.0, "byte")
    w["glue"] = (T * L * q.d_model * 8.0, "byte")
    w["commit"] = (0.0, "byte")
    return w


def aggregate_over_ranks(ms, toks, dist, device):
    """Whole-job figures of independent replicas: the slowest rank's device time, the sum of the tokens."""
    import torch
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    k = torch.tensor([float(toks)], device=device, dtype=torch.float64)
    dist.all_reduce(k, op=dist.ReduceOp.SUM)
    return float(t.item()), int(k.item())


def replica_prompt_seed(base_seed: int, rank: int, generation: int) -> int:
    """Every replica (rank) and every generation of a replica gets its own prompt."""
    return base_seed + 1000 * rank + generation


def make_models(wl, device):
    import paper_2408_05636_b200 as sdd
    wp = synth.model_weights(wl.target, wl.weight_seed, wl.dtype)
    wq = synth.model_weights(wl.drafter, wl.weight_seed, wl.dtype)
    dp = sdd.DeviceModel(wl.target, wp, synth.tensor_names(wl.target), wl.dtype, device)
    dq = sdd.DeviceModel(wl.drafter, wq, synth.tensor_names(wl.drafter), wl.dtype, device)
    return wp, wq, dp, dq


# ----------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import paper_2408_05636_b200 as sdd

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))
    peaks = load_peaks()
    wl = synth.WORKLOADS[args.workload]
    if args.gamma or args.T:
        wl = synth.scaled_workload(wl, gamma=args.gamma or wl.gamma, T=args.T or wl.T)
    if args.workload != WORKLOAD and not args.rounds_only:
        raise SystemExit("other workloads than the headline one are timed with --rounds-only")
    wp, wq, dp, dq = make_models(wl, device)
    V = wl.target.vocab

    gen_idx = [0]

    def new_session():
        seed = replica_prompt_seed(wl.prompt_seed, rank, gen_idx[0])
        gen_idx[0] += 1
        prompts = synth.prompt_ids(V, wl.batch, wl.prompt_len, seed)
        s = sdd.Session(dp, dq, prompts, [wl.prompt_len] * wl.batch, wl.gamma, wl.T, wl.max_new, 1.0, 1.0,
                        wl.philox_seed + gen_idx[0], device)
        s.sdd_sync_status()
        return s

    def next_generation(s):
        """The next request on the same context: new prompt, graphs and workspace kept (sdd_reset)."""
        seed = replica_prompt_seed(wl.prompt_seed, rank, gen_idx[0])
        gen_idx[0] += 1
        s.sdd_reset(synth.prompt_ids(V, wl.batch, wl.prompt_len, seed), [wl.prompt_len] * wl.batch)
        s.sdd_sync_status()

    def emitted(s):
        """(total, minimum over the batch) of the tokens generated so far"""
        e = s.tap_numpy(sdd.TAP_N_EMITTED)
        return int(e.sum()), int(e.min())

    def run_rounds(n, timed):
        """Runs n rounds (across generations if needed).  Returns (device ms, tokens, launches)."""
        nonlocal sess
        ms_total, tok_total, launch_total, left = 0.0, 0, 0, n
        while left > 0:
            e0, emin = emitted(sess)
            if emin >= wl.max_new:
                next_generation(sess)
                e0 = 0
            # rounds this generation can still take: stop a segment when it completes
            _, l0 = sess.sdd_counters()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            ev0.record(sess.stream)
            done = 0
            while done < left:
                sess.sdd_step()
                done += 1
                _, em = sess.sdd_progress()
                if em >= wl.max_new:
                    break
            ev1.record(sess.stream)
            torch.cuda.synchronize()
            sess.sdd_sync_status()
            _, l1 = sess.sdd_counters()
            # rounds enqueued after the generation completed emit nothing but still ran: they are counted
            ms_total += ev0.elapsed_time(ev1)
            tok_total += emitted(sess)[0] - e0
            launch_total += l1 - l0
            left -= done
        return ms_total, tok_total, launch_total

    # One context serves generation after generation, as a server would run it.  Its first generation is untimed: a
    # round's launches are captured into a CUDA graph the first time a padded row count occurs (three counts over a
    # generation of the headline workload), and a capture inside the timed region would stall the device for tens of
    # milliseconds, by an amount that depends on the host's load.  Then W warm-up rounds, then the K timed rounds.
    sess = new_session()
    while emitted(sess)[1] < wl.max_new:
        sess.sdd_step()
    sess.sdd_sync_status()
    next_generation(sess)
    run_rounds(args.warmup, False)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = ClockSampler(local) if rank == 0 else None
    ms, toks, launches = run_rounds(args.steps, True)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        ms, toks = aggregate_over_ranks(ms, toks, dist, device)
    # keep the GPU busy a little longer so that the clock sampler sees load (same work, untimed)
    t_end = time.time() + (0.0 if args.rounds_only else 1.0)
    while time.time() < t_end:
        run_rounds(4, False)
    clock_info = clocks.stop() if clocks else None
    value = toks / (ms * 1e-3)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    if args.rounds_only:
        print(json.dumps({"metric": METRIC, "workload": wl.name, "batch": wl.batch, "gamma": wl.gamma, "T": wl.T,
                          "value": round(value, 2), "unit": UNIT, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4), "gpu_launches": int(launches),
                          "note": "rounds only"}))
        return

    # ---- profiled pass: per-category device time of the same rounds ---------------------------
    sess.close()
    gen_idx[0] = 0
    sess = new_session()
    prof_rounds = min(args.steps, 32)
    cat_ms = {n: 0.0 for n in sdd.PROF_NAMES}
    cat_n = {n: 0 for n in sdd.PROF_NAMES}
    cat_work = {n: 0.0 for n in sdd.PROF_NAMES}
    kinds = {}
    acc_stats = {"accepted": 0, "tested": 0, "ratio_sum": 0.0}
    for _ in range(prof_rounds):
        if emitted(sess)[1] >= wl.max_new:
            sess.close()
            sess = new_session()
        c = int(sess.tap_numpy(sdd.TAP_CTX_LEN)[0])
        sess.sdd_profile_begin()
        sess.sdd_step()
        res = sess.sdd_profile_end()
        n_acc = int(sess.tap_numpy(sdd.TAP_N_ACCEPT)[0])
        tested = n_acc + 1 if n_acc < wl.gamma else wl.gamma
        acc_stats["accepted"] += n_acc
        acc_stats["tested"] += tested
        acc_stats["ratio_sum"] += float(sess.tap_numpy(sdd.TAP_ACCEPT_PROB)[:tested].sum())
        work = round_work(wl, c)
        for n, (m, k) in res.items():
            cat_ms[n] += m
            cat_n[n] += k
            cat_work[n] += work[n][0]
            kinds[n] = work[n][1]
    total_ms = sum(cat_ms.values())
    kernels = {}
    for n in sdd.PROF_NAMES:
        if cat_n[n] == 0:
            continue
        secs = cat_ms[n] * 1e-3
        if kinds[n] == "flop":
            ach, peak, unit, bound = cat_work[n] / secs / 1e12, peaks["tf_sustained"], "TFLOP/s", "tensor"
        else:
            ach, peak, unit, bound = cat_work[n] / secs / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
        kernels[n] = {"share": round(cat_ms[n] / total_ms, 4), "launches": cat_n[n],
                      "avg_us": round(cat_ms[n] * 1e3 / cat_n[n], 2), "bound": bound, "achieved": round(ach, 3),
                      "peak": peak, "unit": unit, "frac": round(ach / peak, 5)}
    # DRAM bytes per launch of the drafter's GEMMs from the ncu capture summarised in
    # profiles/gemm_drafter_traffic_small_bf16.txt (mean of the four GEMMs of a block; valid for the headline workload
    # and for the GEMM kernel as captured)
    traffic_bytes = {"gemm_drafter": 4.62e6} if wl.name == WORKLOAD and not (args.gamma or args.T) else {}
    dom = max(kernels, key=lambda n: kernels[n]["share"])
    roofline = {"kernel": dom, "bound": kernels[dom]["bound"], "achieved": kernels[dom]["achieved"],
                "peak": kernels[dom]["peak"], "unit": kernels[dom]["unit"], "frac": kernels[dom]["frac"],
                "traffic": traffic_bytes.get(dom), "traffic_unit": "bytes per launch (ncu dram read + write)",
                "algorithmic_flops_per_launch": round(cat_work[dom] / max(1, cat_n[dom])),
                "peak_source": f"of {peaks['source']}",
                "timing": f"CUDA-event pairs around every launch in a separate pass of {prof_rounds} rounds"}
    sess.close()

    # ---- the paper's closed forms next to the measurement (Eq. 2, Eq. 3) and the autoregressive context line ----
    alpha_hat = acc_stats["accepted"] / max(1, acc_stats["tested"])
    mean_min = acc_stats["ratio_sum"] / max(1, acc_stats["tested"])   # E_x~q min(1, p/q) = sum_x min(p, q)
    ln_q = wl.T * (2 * wl.drafter.n_layer + 1)
    ln_p = 2 * wl.target.n_layer + 1
    drafter_ms = (cat_ms["gemm_drafter"] + cat_ms["head_drafter"] + cat_ms["attn_drafter"] + cat_ms["sample"] +
                  cat_ms["glue"] + cat_ms["layernorm"] * ln_q / (ln_q + ln_p))
    frac_q = drafter_ms / total_ms
    ms_round = ms / args.steps
    c1 = frac_q * ms_round / wl.T
    c2 = (1.0 - frac_q) * ms_round
    e_tok = (1 - alpha_hat ** (wl.gamma + 1)) / (1 - alpha_hat) if alpha_hat < 1 else wl.gamma + 1
    s_ar = new_session()
    for _ in range(4):
        s_ar.sdd_ar_step()
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ar_steps = 128
    s_ar.stream.synchronize()
    a0.record(s_ar.stream)
    for _ in range(ar_steps):
        s_ar.sdd_ar_step()
    a1.record(s_ar.stream)
    s_ar.sdd_sync_status()
    ar_ms = a0.elapsed_time(a1) / ar_steps
    s_ar.close()
    # speculative decoding with an autoregressive drafter of the same size (the warm start of the paper's
    # "Sequence initialization"), gamma_sps = 5: context line
    wa = synth.model_weights(wl.ar_drafter, wl.ar_weight_seed, wl.dtype)
    da = sdd.DeviceModel(wl.ar_drafter, wa, synth.tensor_names(wl.ar_drafter), wl.dtype, device)
    s_sps = new_session()
    s_sps.sdd_sps_attach(da)
    g_sps, sps_rounds = 5, 32
    for _ in range(4):
        s_sps.sdd_sps_step(g_sps)
    s_sps.sdd_sync_status()
    e_sps0 = emitted(s_sps)[0]
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record(s_sps.stream)
    for _ in range(sps_rounds):
        s_sps.sdd_sps_step(g_sps)
    b1.record(s_sps.stream)
    s_sps.sdd_sync_status()
    sps_ms = b0.elapsed_time(b1)
    sps_tok = emitted(s_sps)[0] - e_sps0
    s_sps.close()
    model = {"alpha_hat": round(alpha_hat, 4), "mean_sum_min_pq": round(mean_min, 4),
             "tokens_per_round_eq2": round(e_tok, 3), "tokens_per_round_measured": round(toks / args.steps / world, 3),
             "c1_ms_per_drafter_evaluation": round(c1, 4), "c2_ms_target_and_accept": round(c2, 4),
             "tokens_per_s_eq3": round(e_tok / ((wl.T * c1 + c2) * 1e-3), 1),
             "autoregressive_target_tokens_per_s": round(1e3 / ar_ms, 1),
             "sps_warm_start_tokens_per_s": round(sps_tok / (sps_ms * 1e-3), 1),
             "sps_warm_start_ms_per_round": round(sps_ms / sps_rounds, 4),
             "sps_warm_start_gamma": g_sps,
             "note": "Eq. 2 / Eq. 3 of the paper with the measured acceptance rate and stage times; the autoregressive line "
                     "is plain decoding of the same synthetic target (sdd_ar_step) and the sps lines are standard speculative "
                     "decoding with an autoregressive drafter of the drafter's size (sdd_sps_step), context only"}

    # ---- stand-alone kernels (paper_2408_05636_b200.microbench) --------------------------------
    from paper_2408_05636_b200 import microbench
    rows, g4 = 64, 32
    acc = microbench.accept(rows, g4, V, 0.5, iters=20, warmup=3)
    accept_roof = {"bound": "hbm", "achieved": round(acc["gbs"], 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                   "frac": round(acc["gbs"] / peaks["hbm_gbs"], 4),
                   # ncu capture of the 16-row case scaled by 4 (profiles/accept_kernels_16x32x50257.txt): statistics pass
                   # 209.08 + 3.7 MB, acceptance pass 6.69 MB per 16 rows; algorithmic bytes 836.3 MB
                   "traffic": round(4 * (209.08e6 + 3.7e6 + 6.69e6)), "traffic_unit": "bytes per call (two launches)",
                   "ms": round(acc["us"] * 1e-3, 4),
                   "launches_per_call": 2,
                   "workload": f"{rows} rows x gamma {g4} x V {V} fp32 logits, inputs 0.84 GB > L2",
                   "mean_accepted": acc["mean_accepted"], "peak_source": f"of {peaks['source']}"}
    gm = microbench.gemm(16384, 4096, 1024, epilogue=1, iters=20, warmup=3)
    gemm_roof = {"bound": "tensor", "achieved": round(gm["tflops"], 1), "peak": peaks["tf_burst"], "unit": "TFLOP/s",
                 "frac": round(gm["tflops"] / peaks["tf_burst"], 4), "traffic": None, "us": round(gm["us"], 2),
                 "workload": "bf16 GEMM 16384 x 4096 x 1024 with bias + GELU epilogue (drafter FC1 at batch 16), timed alone",
                 "peak_source": f"of {peaks['source']} (burst)"}

    # ---- end to end through the C ABI with host buffers ----------------------------------------
    # One context serves generation after generation (sdd_reset), as a server would: the first, untimed generation
    # captures the round graphs; the timed one starts with the prompt in pinned host memory (H2D + prefill inside the
    # timed region).  The emitted ids of every round land in pinned host buffers (written by the commit kernel over the
    # bus) and are consumed by the host as soon as sdd_progress counts the round, while the next round is already
    # enqueued (two output buffers in alternation).
    host_out = [torch.full((wl.gamma + 2,), -1, dtype=torch.int32).pin_memory() for _ in range(2)]

    def e2e_generation(s):
        enq = seen = got = 0
        generated = []
        while got < wl.max_new:
            while enq < seen + 2:
                hb = host_out[enq % 2]
                s.sdd_step(hb[: wl.gamma + 1], hb[wl.gamma + 1:])
                enq += 1
            while s.sdd_progress()[0] <= seen:
                pass
            hb = host_out[seen % 2]
            n = int(hb[wl.gamma + 1])
            generated += hb[:n].tolist()
            got += n
            seen += 1
        s.sdd_sync_status()
        return got, seen, generated

    warm_prompt = synth.prompt_ids(V, 1, wl.prompt_len, wl.prompt_seed + 77)
    s = sdd.Session(dp, dq, warm_prompt, [wl.prompt_len], wl.gamma, wl.T, wl.max_new, 1.0, 1.0, wl.philox_seed, device)
    e2e_generation(s)
    pinned_prompt = torch.from_numpy(synth.prompt_ids(V, 1, wl.prompt_len, wl.prompt_seed)).pin_memory()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    s.sdd_reset(pinned_prompt.numpy(), [wl.prompt_len])
    got, rounds, generated = e2e_generation(s)
    t1 = time.perf_counter()
    s.close()
    e2e = {"value": round(got / (t1 - t0), 2), "unit": UNIT,
           "h2d_bytes_per_step": round(wl.prompt_len * 4 / rounds, 1), "d2h_bytes_per_step": (wl.gamma + 2) * 4,
           "includes": "sdd_reset (prompt H2D from pinned memory, prefill), every round, the emitted ids of every round "
                       "written to pinned host memory by the commit kernel and read by the host round by round; the context "
                       "and its round graphs come from an earlier, untimed generation",
           "rounds": rounds}

    # ---- the oracle on the host cores, bounded sample -------------------------------------------
    cpu = time_oracle(wl, wp, wq, budget_s=20.0, max_rounds=3)

    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": CONFIG,
        "tokens_per_step": round(toks / args.steps / world, 3),
        "clocks": clock_info, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "roofline_accept_kernel": accept_roof, "roofline_gemm_kernel": gemm_roof,
        "kernels": kernels, "paper_model": model, "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------------
def time_oracle(wl, wp, wq, budget_s, max_rounds):
    from oracle import specdiff as sd
    from oracle.transformer import Model
    mp, mq = Model(wl.target, wp), Model(wl.drafter, wq)
    prompt = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)[0]
    ids = [int(x) for x in prompt]
    t0 = time.perf_counter()
    rounds = 0
    while rounds < max_rounds and (rounds == 0 or (time.perf_counter() - t0) * (rounds + 1) / rounds < budget_s):
        tr = sd.specdiff_round(mp, mq, np.array(ids), wl.gamma, wl.T, 1.0, 1.0, wl.philox_seed, rounds)
        ids += tr.emitted
        rounds += 1
    dt = time.perf_counter() - t0
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count()
    return {"value": round((len(ids) - len(prompt)) / dt, 3), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {rounds} round(s) of the same generation (numpy fp64), {dt:.1f} s",
            "s_per_round": round(dt / rounds, 3)}


def run_reference(args):
    """The CPU oracle as it stands, on the host cores; each step is one oracle round of the same workload.
    Rounds stop early when a time budget of about three minutes is used up."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import specdiff as sd
    from oracle.transformer import Model
    wl = synth.WORKLOADS[WORKLOAD]
    wp = synth.model_weights(wl.target, wl.weight_seed, wl.dtype)
    wq = synth.model_weights(wl.drafter, wl.weight_seed, wl.dtype)
    mp, mq = Model(wl.target, wp), Model(wl.drafter, wq)
    prompt = synth.prompt_ids(wl.target.vocab, 1, wl.prompt_len, wl.prompt_seed)[0]
    ids = [int(x) for x in prompt]
    budget = 180.0
    t_start = time.perf_counter()
    rnd = 0
    for _ in range(args.warmup):
        if time.perf_counter() - t_start > 0.25 * budget:
            break
        ids += sd.specdiff_round(mp, mq, np.array(ids), wl.gamma, wl.T, 1.0, 1.0, wl.philox_seed, rnd).emitted
        rnd += 1
    t0 = time.perf_counter()
    done, toks = 0, 0
    while done < args.steps:
        em = sd.specdiff_round(mp, mq, np.array(ids), wl.gamma, wl.T, 1.0, 1.0, wl.philox_seed, rnd).emitted
        ids += em
        toks += len(em)
        rnd += 1
        done += 1
        if time.perf_counter() - t_start > budget:
            break
    dt = time.perf_counter() - t0
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count()
    value = toks / dt
    sample = f"{done} oracle round(s) of the same generation (numpy fp64) in {dt:.1f} s"
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": done, "steps_requested": args.steps,
            "warmup": args.warmup, "ms_per_step": round(dt * 1e3 / done, 2), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": CONFIG,
            "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(synth.WORKLOADS),
                    help="with --rounds-only: time another configuration (default: the headline one)")
    ap.add_argument("--gamma", type=int, default=0)
    ap.add_argument("--T", type=int, default=0)
    ap.add_argument("--rounds-only", action="store_true",
                    help="run only the warm-up and timed rounds and print a short line (for profiler captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 12 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 64 if args.steps is None else args.steps
        args.warmup = max(3, 8 if args.warmup is None else args.warmup)
        run_ours(args)


if __name__ == "__main__":
    main()
