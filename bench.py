#!/usr/bin/env python
"""Benchmark of the SpecDiff draft–verify–accept round on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one whole round (T drafter evaluations, one target verification, acceptance, commit).
The headline workload is the largest batch-1 configuration: the GPT-2-XL-shaped bf16 target (48L d1600) with the
24L d1024 masked-diffusion drafter, V = 50257, prompt 512 random ids, gamma = 32, T = 16, 512 new tokens.  When a
generation reaches its 512 tokens the next one (next prompt seed) starts on the same context (sdd_reset); set-up,
the context's first generation (which captures the round graphs) and prefill are outside the timed segments.
Rank 0 also reports, as nested records of the same JSON line: the GPT-2-small-shaped pair (gamma 16, T 8) and one
point of the batch-16 serving sweep, the acceptance kernels alone over draft lengths 8..128, one large GEMM alone,
the end-to-end figure through the C ABI with host buffers, and the CPU oracle on a bounded sample.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

WORKLOAD = "xl_bf16"
METRIC = "SpecDiff generated tokens/s at bs=1"
UNIT = "tokens/s"


def describe(wl) -> str:
    p, q = wl.target, wl.drafter
    return (f"bf16 {p.n_layer}L d{p.d_model} target + {q.n_layer}L d{q.d_model} masked-diffusion drafter, V={p.vocab}, "
            f"prompt {wl.prompt_len}, gamma={wl.gamma}, T={wl.T}, batch {wl.batch}, {wl.max_new} new tokens")


def config_of(wl):
    weights_mb = (12 * wl.target.d_model ** 2 * wl.target.n_layer + 12 * wl.drafter.d_model ** 2 * wl.drafter.n_layer) * 2 / 1e6
    return {"workload": describe(wl),
            "l2": f"no flush: consecutive rounds of one generation; each round streams about {weights_mb / 1e3:.1f} GB of "
                  "block weights per network pass (> 126 MB L2)",
            "graphs": "one context serves all generations (sdd_reset); its first, untimed generation captures the round graphs",
            "multi_gpu": "independent replicas, no collective on the data path"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "tf_burst": d["bf16_tflops"], "tf_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


def profile_value(fname: str, key: str):
    """A figure of a committed ncu summary: the line `key = number` of profiles/<fname> (None if absent)."""
    try:
        txt = open(os.path.join(ROOT, "profiles", fname)).read()
    except OSError:
        return None
    m = re.search(r"^\s*" + re.escape(key) + r"\s*=\s*([0-9.eE+-]+)", txt, flags=re.M)
    return float(m.group(1)) if m else None


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
#   c = context length, evals = drafter evaluations that actually ran in the round (skipped ones do no work)
# ----------------------------------------------------------------------------------------------
def round_work(wl, c: float, evals: float):
    q, p = wl.drafter, wl.target
    G, V, B = wl.gamma, p.vocab, wl.batch
    L = c + G
    w = {}
    w["gemm_drafter"] = (B * evals * 2.0 * L * 12 * q.d_model ** 2 * q.n_layer, "flop")
    # the LM heads stream the tied embedding once per evaluation for gamma (+1) rows: weight-bound like the target's GEMMs
    w["head_drafter"] = (evals * (V * q.d_model * 2.0 + B * G * V * 4.0), "byte")
    w["attn_drafter"] = (B * evals * 4.0 * L * L * q.d_model * q.n_layer, "flop")
    w["gemm_target"] = (12.0 * p.d_model ** 2 * p.n_layer * 2, "byte")              # weights streamed once
    w["head_target"] = (V * p.d_model * 2.0 + B * (G + 1) * V * 4.0, "byte")
    w["attn_target"] = (B * 2.0 * p.n_layer * c * p.d_model * 2, "byte")            # K and V of the cache
    w["row_stats"] = (B * (G + 1) * V * 4.0, "byte")
    w["accept"] = (B * 4.0 * V * 4, "byte")                                         # p row twice, q row twice
    w["sample"] = (B * 2.0 * G * V * 4, "byte")
    w["layernorm"] = (B * (evals * (2 * q.n_layer) * L * q.d_model * 6.0 + 2 * p.n_layer * (G + 1) * p.d_model * 6.0), "byte")
    w["glue"] = (B * evals * L * q.d_model * 8.0, "byte")
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


class Runner:
    """One context that serves generation after generation of a workload, as a server would run it."""

    def __init__(self, wl, dp, dq, device, rank):
        self.wl, self.dp, self.dq, self.device, self.rank = wl, dp, dq, device, rank
        self.gen = 0
        self.sess = None

    def _prompts(self):
        seed = replica_prompt_seed(self.wl.prompt_seed, self.rank, self.gen)
        self.gen += 1
        return synth.prompt_ids(self.wl.target.vocab, self.wl.batch, self.wl.prompt_len, seed)

    def open(self):
        import paper_2408_05636_b200 as sdd
        wl = self.wl
        self.sess = sdd.Session(self.dp, self.dq, self._prompts(), [wl.prompt_len] * wl.batch, wl.gamma, wl.T, wl.max_new,
                                1.0, 1.0, wl.philox_seed + self.gen, self.device)
        self.sess.sdd_sync_status()
        return self

    def next_generation(self):
        """The next request on the same context: new prompt, graphs and workspace kept (sdd_reset)."""
        self.sess.sdd_reset(self._prompts(), [self.wl.prompt_len] * self.wl.batch)
        self.sess.sdd_sync_status()

    def emitted(self):
        """(total, minimum over the batch) of the tokens generated so far"""
        import paper_2408_05636_b200 as sdd
        e = self.sess.tap_numpy(sdd.TAP_N_EMITTED)
        return int(e.sum()), int(e.min())

    def evals(self):
        import paper_2408_05636_b200 as sdd
        e = self.sess.tap_numpy(sdd.TAP_EVALS)
        return int(e[0]), int(e[1])

    def first_generation(self):
        """The context's first generation, untimed: a round's launches are captured into a CUDA graph the first time
        a padded row count occurs, and a capture inside a timed region would stall the device for tens of
        milliseconds, by an amount that depends on the host's load."""
        while self.emitted()[1] < self.wl.max_new:
            for _ in range(8):
                self.sess.sdd_step()
        self.sess.sdd_sync_status()
        self.next_generation()

    def run_rounds(self, n):
        """Runs n rounds (across generations if needed).  Returns (device ms, tokens, launches, evaluations run,
        evaluations skipped, mean context length)."""
        import torch
        sess, wl = self.sess, self.wl
        ms_total, tok_total, launch_total, run_total, skip_total, left = 0.0, 0, 0, 0, 0, n
        ctx_sum = 0.0
        while left > 0:
            e0, emin = self.emitted()
            if emin >= wl.max_new:
                self.next_generation()
                e0 = 0
            r0, s0 = self.evals()
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
            r1, s1 = self.evals()
            e1 = self.emitted()[0]
            # rounds enqueued after the generation completed emit nothing but still ran: they are counted
            ms_total += ev0.elapsed_time(ev1)
            tok_total += e1 - e0
            launch_total += l1 - l0
            run_total += r1 - r0
            skip_total += s1 - s0
            ctx_sum += done * (wl.prompt_len + (e0 + e1) / (2.0 * wl.batch))
            left -= done
        return ms_total, tok_total, launch_total, run_total, skip_total, ctx_sum / n

    def close(self):
        if self.sess is not None:
            self.sess.close()
            self.sess = None


def profile_rounds(runner, n_rounds, peaks):
    """Per-category device time of n_rounds rounds (CUDA-event pairs around every launch, recorded inside a one-off
    graph of each round) -> (table, totals)."""
    import paper_2408_05636_b200 as sdd
    wl, sess = runner.wl, runner.sess
    cat_ms = {n: 0.0 for n in sdd.PROF_NAMES}
    cat_n = {n: 0 for n in sdd.PROF_NAMES}
    cat_work = {n: 0.0 for n in sdd.PROF_NAMES}
    kinds = {}
    acc = {"accepted": 0, "tested": 0, "ratio_sum": 0.0}
    for _ in range(n_rounds):
        if runner.emitted()[1] >= wl.max_new:
            runner.next_generation()
        c = float(sess.tap_numpy(sdd.TAP_CTX_LEN).mean())
        r0, _ = runner.evals()
        sess.sdd_profile_begin()
        sess.sdd_step()
        res = sess.sdd_profile_end()
        r1, _ = runner.evals()
        n_acc = sess.tap_numpy(sdd.TAP_N_ACCEPT)
        prob = sess.tap_numpy(sdd.TAP_ACCEPT_PROB).reshape(wl.batch, wl.gamma)
        for b in range(wl.batch):
            na = int(n_acc[b])
            tested = na + 1 if na < wl.gamma else wl.gamma
            acc["accepted"] += na
            acc["tested"] += tested
            acc["ratio_sum"] += float(prob[b, :tested].sum())
        work = round_work(wl, c, r1 - r0)
        for n, (m, k) in res.items():
            cat_ms[n] += m
            cat_n[n] += k
            cat_work[n] += work[n][0]
            kinds[n] = work[n][1]
    total_ms = sum(cat_ms.values())
    kernels = {}
    for n in sdd.PROF_NAMES:
        if cat_n[n] == 0 or cat_ms[n] <= 0.0:
            continue
        secs = cat_ms[n] * 1e-3
        if kinds[n] == "flop":
            ach, peak, unit, bound = cat_work[n] / secs / 1e12, peaks["tf_sustained"], "TFLOP/s", "tensor"
        else:
            ach, peak, unit, bound = cat_work[n] / secs / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
        kernels[n] = {"share": round(cat_ms[n] / total_ms, 4), "launches": cat_n[n],
                      "avg_us": round(cat_ms[n] * 1e3 / cat_n[n], 2), "bound": bound, "achieved": round(ach, 3),
                      "peak": peak, "unit": unit, "frac": round(ach / peak, 5),
                      "work_per_launch": round(cat_work[n] / cat_n[n])}
    return kernels, {"ms": cat_ms, "total_ms": total_ms, "acc": acc}


def rounds_record(wl, dp, dq, device, rank, warmup, steps, pregenerate=True):
    """Timed rounds of another workload on its own context -> a short record (rank 0's nested sub-records)."""
    r = Runner(wl, dp, dq, device, rank).open()
    if pregenerate:
        r.first_generation()
    r.run_rounds(warmup)
    ms, toks, launches, ev_run, ev_skip, ctx = r.run_rounds(steps)
    r.close()
    return {"workload": describe(wl), "ms_per_round": round(ms / steps, 4), "tokens_per_s": round(toks / (ms * 1e-3), 2),
            "tokens_per_round": round(toks / steps, 3), "launches_per_round": round(launches / steps, 1),
            "evaluations_run_per_round": round(ev_run / steps, 2), "evaluations_skipped_per_round": round(ev_skip / steps, 2),
            "rounds": steps, "mean_context": round(ctx, 1)}


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

    runner = Runner(wl, dp, dq, device, rank).open()
    if not args.fresh:
        runner.first_generation()
    runner.run_rounds(args.warmup)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = ClockSampler(local) if rank == 0 else None
    ms, toks, launches, ev_run, ev_skip, ctx_mean = runner.run_rounds(args.steps)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        ms, toks = aggregate_over_ranks(ms, toks, dist, device)
    # keep the GPU busy a little longer so that the clock sampler sees load (same work, untimed)
    t_end = time.time() + (0.0 if args.rounds_only else 1.0)
    while time.time() < t_end:
        runner.run_rounds(4)
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
                          "evaluations_run": ev_run, "evaluations_skipped": ev_skip, "note": "rounds only"}))
        return

    # ---- one whole generation on the same context (steadier than a window of K rounds) ---------------------------
    runner.next_generation()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    g0.record(runner.sess.stream)
    gen_rounds = 0
    while True:
        runner.sess.sdd_step()
        gen_rounds += 1
        if runner.sess.sdd_progress()[1] >= wl.max_new:
            break
    g1.record(runner.sess.stream)
    torch.cuda.synchronize()
    runner.sess.sdd_sync_status()
    gen_ms = g0.elapsed_time(g1)
    whole_generation = {"tokens_per_s": round(runner.emitted()[0] / (gen_ms * 1e-3), 2), "rounds_enqueued": gen_rounds,
                        "ms": round(gen_ms, 2), "tokens": runner.emitted()[0],
                        "note": "prefill excluded; rounds enqueued after the last token was committed are included"}

    # ---- profiled pass: per-category device time of rounds of the same workload -------------------------------
    runner.next_generation()
    prof_rounds = max(2, min(args.steps, 6))
    kernels, tot = profile_rounds(runner, prof_rounds, peaks)
    total_ms, cat_ms, acc_stats = tot["total_ms"], tot["ms"], tot["acc"]
    dom = max(kernels, key=lambda n: kernels[n]["share"])
    # DRAM bytes per launch of the dominant category from the committed ncu summary of this workload (if there is one)
    traffic = profile_value(f"{dom}_traffic_{wl.name}.txt", "dram_bytes_per_launch") if not (args.gamma or args.T) else None
    compact = {n: {"share": k["share"], "avg_us": k["avg_us"], "launches_per_round": round(k["launches"] / prof_rounds, 1),
                   "achieved": k["achieved"], "unit": k["unit"], "frac": k["frac"]} for n, k in kernels.items()}
    roofline = {"kernel": dom, "bound": kernels[dom]["bound"], "achieved": kernels[dom]["achieved"],
                "peak": kernels[dom]["peak"], "unit": kernels[dom]["unit"], "frac": kernels[dom]["frac"],
                "traffic": traffic, "traffic_unit": "bytes per launch (ncu dram read + write)",
                "algorithmic_work_per_launch": kernels[dom]["work_per_launch"],
                "peak_source": f"of {peaks['source']} (sustained bf16 for flop-bound rows, copy bandwidth for byte-bound rows)",
                "timing": f"CUDA-event pairs around every launch in a separate pass of {prof_rounds} rounds; work counted "
                          "only for drafter evaluations that ran",
                "kernels": compact}

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
    runner.close()

    def fresh_session(seed_off):
        prompts = synth.prompt_ids(V, wl.batch, wl.prompt_len, wl.prompt_seed + seed_off)
        s = sdd.Session(dp, dq, prompts, [wl.prompt_len] * wl.batch, wl.gamma, wl.T, wl.max_new, 1.0, 1.0,
                        wl.philox_seed + seed_off, device)
        s.sdd_sync_status()
        return s

    def session_emitted(s):
        return int(s.tap_numpy(sdd.TAP_N_EMITTED).sum())

    s_ar = fresh_session(301)
    for _ in range(4):
        s_ar.sdd_ar_step()
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ar_steps = 96
    s_ar.stream.synchronize()
    a0.record(s_ar.stream)
    for _ in range(ar_steps):
        s_ar.sdd_ar_step()
    a1.record(s_ar.stream)
    s_ar.sdd_sync_status()
    ar_ms = a0.elapsed_time(a1) / ar_steps
    s_ar.close()
    # speculative decoding with an autoregressive drafter of the drafter's size (the warm start of the paper's
    # "Sequence initialization"), gamma_sps = 5: context line
    wa = synth.model_weights(wl.ar_drafter, wl.ar_weight_seed, wl.dtype)
    da = sdd.DeviceModel(wl.ar_drafter, wa, synth.tensor_names(wl.ar_drafter), wl.dtype, device)
    del wa
    s_sps = fresh_session(302)
    s_sps.sdd_sps_attach(da)
    g_sps, sps_rounds = 5, 24
    for _ in range(4):
        s_sps.sdd_sps_step(g_sps)
    s_sps.sdd_sync_status()
    e_sps0 = session_emitted(s_sps)
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    b0.record(s_sps.stream)
    for _ in range(sps_rounds):
        s_sps.sdd_sps_step(g_sps)
    b1.record(s_sps.stream)
    s_sps.sdd_sync_status()
    sps_ms = b0.elapsed_time(b1)
    sps_tok = session_emitted(s_sps) - e_sps0
    s_sps.close()
    del da
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

    s = fresh_session(77)
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

    # ---- the batch-16 serving point on the same weights (one point of the sweep) --------------------------------
    wl16 = synth.WORKLOADS["xl_bf16_b16"]
    try:
        serving = rounds_record(wl16, dp, dq, device, rank, warmup=3, steps=6, pregenerate=False)
        serving["note"] = ("gamma 16, T 8, 16 prompts of 1024 ids on this run's XL weights; rounds 4-9 of a generation "
                           "(one padded row count, its graph captured by the warm-up rounds)")
    except Exception as exc:   # reported, not fatal: the headline figures above stand on their own
        serving = {"workload": describe(wl16), "error": str(exc)[:200]}

    # ---- the oracle on the host cores, bounded sample (before the weights are dropped) ---------------------------
    cpu = time_oracle_sample(wl, wp, wq, toks / args.steps / world)
    del dp, dq, wp, wq
    torch.cuda.empty_cache()

    # ---- the GPT-2-small-shaped pair (gamma 16, T 8) ------------------------------------------------------------
    wls = synth.WORKLOADS["small_bf16"]
    try:
        _, _, dps, dqs = make_models(wls, device)
        small = rounds_record(wls, dps, dqs, device, rank, warmup=8, steps=64)
        del dps, dqs
    except Exception as exc:
        small = {"workload": describe(wls), "error": str(exc)[:200]}
    torch.cuda.empty_cache()

    # ---- stand-alone kernels (paper_2408_05636_b200.microbench) --------------------------------
    from paper_2408_05636_b200 import microbench
    rows, g4 = 64, 32
    base = synth.accept_case(rows, g4, V, 0.5, seed=31)     # the case tests/test_gpu_accept.py checks row by row
    sweep = {}
    for g in (8, 16, 32, 64, 128):
        r = microbench.accept_case_timed(base, g, iters=20, warmup=3)
        sweep[str(g)] = {"us": round(r["us"], 2), "gbs": round(r["gbs"], 1), "frac": round(r["gbs"] / peaks["hbm_gbs"], 4),
                         "mbytes": round(r["bytes"] / 1e6, 1), "mean_accepted": round(r["mean_accepted"], 2)}
    per16 = profile_value("accept_kernels_16x32x50257.txt", "dram_bytes_per_call")
    accept_roof = {"bound": "hbm", "achieved": sweep[str(g4)]["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                   "frac": sweep[str(g4)]["frac"],
                   # ncu capture of the 16-row case (profiles/accept_kernels_16x32x50257.txt), scaled by the rows: the
                   # statistics pass is one CTA per 8192-element chunk, traffic grows in proportion to the rows
                   "traffic": round(per16 * rows / 16) if per16 else None,
                   "traffic_unit": "bytes per call (two launches)",
                   "algorithmic_bytes": rows * (2 * g4 + 1) * V * 4,
                   "ms": round(sweep[str(g4)]["us"] * 1e-3, 4), "launches_per_call": 2,
                   "workload": f"{rows} rows x gamma {g4} x V {V} fp32 logits from synth.accept_case(seed 31), inputs 0.84 GB > L2",
                   "sweep_gamma": sweep, "peak_source": f"of {peaks['source']}"}
    del base
    gm = microbench.gemm(16384, 4096, 1024, epilogue=1, iters=20, warmup=3)
    gemm_roof = {"bound": "tensor", "achieved": round(gm["tflops"], 1), "peak": peaks["tf_burst"], "unit": "TFLOP/s",
                 "frac": round(gm["tflops"] / peaks["tf_burst"], 4), "traffic": None, "us": round(gm["us"], 2),
                 "workload": "bf16 GEMM 16384 x 4096 x 1024 with bias + GELU epilogue (drafter FC1 at batch 16), timed alone",
                 "peak_source": f"of {peaks['source']} (burst)"}
    roofline["accept"] = accept_roof
    roofline["gemm"] = gemm_roof
    # what the acceptance step of a round reads, next to the size of the target's logit matrix: the soft-max statistics
    # come out of the LM head's epilogue (one pair per row and 128-row slice of the vocabulary), so the acceptance kernel
    # reads those pairs, gamma target logits at the draft ids, and the target and draft rows of the first rejection twice
    pairs = (V + 127) // 128
    roofline["accept_path_in_round"] = {
        "bytes_read_per_round": (wl.gamma + 1) * pairs * 8 + 4 * V * 4 + wl.gamma * 4,
        "logit_matrix_bytes": (wl.gamma + 1) * V * 4,
        "row_stats_launches_per_round": round(kernels["row_stats"]["launches"] / prof_rounds, 2) if "row_stats" in kernels else 0,
        "note": "the logit matrix is written once by the LM head and never read in full"}

    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_of(wl),
        "tokens_per_step": round(toks / args.steps / world, 3),
        "evaluations_per_step": {"run": round(ev_run / args.steps, 2), "skipped": round(ev_skip / args.steps, 2)},
        "clocks": clock_info, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "cpu_baseline": cpu,
        "whole_generation": whole_generation,
        "other_configs": {"small_bf16": small, "xl_bf16_b16": serving},
        "kernels": kernels, "paper_model": model,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------------
def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count()


def time_oracle_sample(wl, wp, wq, tokens_per_round):
    """The oracle's round of the headline workload costs minutes on the host cores (T drafter evaluations of 24 layers
    over 544 positions, then a 48-layer causal forward), so a bounded sample is timed: ONE drafter evaluation, the
    target's verification forward and the acceptance step of the first round, scaled to a round as
    T * t_evaluation + t_verify + t_accept."""
    from oracle import specdiff as sd
    from oracle.transformer import Model, drafter_slot_logits, target_verify_logits
    mp, mq = Model(wl.target, wp), Model(wl.drafter, wq)
    V = wl.target.vocab
    ctx = synth.prompt_ids(V, 1, wl.prompt_len, wl.prompt_seed)[0].astype(np.int64)
    t0 = time.perf_counter()
    st = sd.DraftState.fresh(wl.gamma, V)
    lg = drafter_slot_logits(mq, ctx, st.slots)
    sd.unmask_sample_step(st, lg, 1, 1.0, wl.philox_seed, 0, 0)          # k = 1 reveals every slot
    t1 = time.perf_counter()
    lam = target_verify_logits(mp, ctx, st.slots)
    t2 = time.perf_counter()
    sd.accept_resample(lam, st.qrows, st.logq, st.slots, 1.0, 1.0, wl.philox_seed, 0, 0)
    t3 = time.perf_counter()
    round_s = wl.T * (t1 - t0) + (t2 - t1) + (t3 - t2)
    return {"value": round(tokens_per_round / round_s, 4), "unit": UNIT, "cores": host_cores(), "kind": "oracle",
            "sample": f"one of the {wl.T} drafter evaluations ({t1 - t0:.1f} s), the verification forward ({t2 - t1:.1f} s) and "
                      f"the acceptance step ({t3 - t2:.2f} s) of the first round (numpy fp64); scaled to a round as "
                      f"T * evaluation + verification + acceptance = {round_s:.0f} s, with the device run's "
                      f"{tokens_per_round:.2f} tokens per round",
            "s_per_round": round(round_s, 1)}


def run_reference(args):
    """The CPU oracle as it stands, on the host cores; each step is one whole oracle round of the headline workload
    (about two minutes each on 16 cores), so the rounds stop when a budget of about five minutes is used up; no
    warm-up round is run when one round alone takes a quarter of the budget."""
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
    budget = 300.0
    t_start = time.perf_counter()
    rnd = 0
    done, toks, dt, warm = 0, 0, 0.0, 0
    per_round = None
    while done < args.steps:
        t0 = time.perf_counter()
        em = sd.specdiff_round(mp, mq, np.array(ids), wl.gamma, wl.T, 1.0, 1.0, wl.philox_seed, rnd).emitted
        t1 = time.perf_counter()
        ids += em
        rnd += 1
        per_round = t1 - t0
        # the first rounds are warm-up only while a round is cheap; a round that costs a quarter of the budget is timed
        if warm < args.warmup and per_round < 0.05 * budget:
            warm += 1
            continue
        dt += per_round
        toks += len(em)
        done += 1
        if time.perf_counter() - t_start + per_round > budget:
            break
    value = toks / dt
    cores = host_cores()
    sample = f"{done} whole oracle round(s) of the same generation (numpy fp64) in {dt:.1f} s, after {warm} warm-up round(s)"
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": done, "steps_requested": args.steps,
            "warmup": warm, "ms_per_step": round(dt * 1e3 / done, 2), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl),
            "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
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
    ap.add_argument("--fresh", action="store_true",
                    help="skip the context's untimed first generation (short profiler captures: the round graphs are then "
                         "captured inside the warm-up rounds)")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 2 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 32 if args.steps is None else args.steps
        args.warmup = max(3, 8 if args.warmup is None else args.warmup)
        run_ours(args)


if __name__ == "__main__":
    main()
