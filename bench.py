#!/usr/bin/env python
"""Rollout-generation benchmark: generated tokens/s on B200 for a named decoder shape.

One "step" is one whole rollout of the workload: prefill of every prompt once, then T-1
decode steps for all P*G sequences, sampling and log-probabilities included.  Inputs are
seeded and synthetic (random-init bf16 weights, uniform token ids).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 8B] [--impl ours|reference]

Prints one JSON line (rank 0).  With --impl reference the CPU oracle is timed instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

# measured DRAM bytes per algorithmic byte of the prefix + suffix launch (ncu, see profiles/): with the
# resident suffix kernel (decode steps below LONG_SUFFIX_STEP) and with one suffix CTA per item (above)
ATTN_DRAM_PER_ALG_BYTE = {"resident": 251.56 / 244.5, "waves": 170.61 / 166.2}
LONG_SUFFIX_STEP = 1088
METRIC = "rollout generated tokens/s"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = f"/tmp/echo_bench_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu_index), "-lms", "200"],
                                         stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    smax.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# algorithmic bytes / flops of the workload (what the method must move, not what the kernels do)
# ---------------------------------------------------------------------------------------------
def model_counts(shape):
    d, hd = shape.d_model, shape.head_dim
    n_layer = d * hd * (2 * shape.n_q_heads + 2 * shape.n_kv_heads) + 3 * d * shape.d_ff
    n_body = shape.n_layers * n_layer
    n_lm = shape.vocab * d
    kv_tok = 2 * shape.n_layers * shape.n_kv_heads * hd * 2          # bytes of K+V per token, all layers
    return n_body, n_lm, kv_tok


def step_bytes_flops(shape, P, G, Lp, i):
    """Decode step i (1-based): weights once, each group's prefix once, each sample's own i
    generated tokens, plus the new token's K/V write."""
    n_body, n_lm, kv_tok = model_counts(shape)
    B = P * G
    byts = 2 * (n_body + n_lm) + kv_tok * (P * Lp + B * i) + kv_tok * B
    flops = 2 * (n_body + n_lm) * B + 4 * shape.n_q_heads * shape.head_dim * shape.n_layers * B * (Lp + i)
    return byts, flops


def attention_bytes(shape, P, G, Lp, i):
    """Algorithmic bytes of ONE layer's decode attention at step i: the group's prefix K/V once,
    each sample's own generated K/V, q in and output out (bf16)."""
    kv_tok_layer = 2 * shape.n_kv_heads * shape.head_dim * 2
    B = P * G
    return kv_tok_layer * (P * Lp + B * i) + 2 * B * shape.n_q_heads * shape.head_dim * 2


def rollout_roofline_seconds(shape, P, G, Lp, T, bw_gbs, tflops):
    n_body, n_lm, kv_tok = model_counts(shape)
    pre_flops = 2 * n_body * P * Lp + 2 * shape.n_q_heads * shape.head_dim * shape.n_layers * P * Lp * Lp
    pre_bytes = 2 * n_body + kv_tok * P * Lp
    t = max(pre_bytes / (bw_gbs * 1e9), pre_flops / (tflops * 1e12))
    for i in range(1, T):
        b, f = step_bytes_flops(shape, P, G, Lp, i)
        t += max(b / (bw_gbs * 1e9), f / (tflops * 1e12))
    return t


# ---------------------------------------------------------------------------------------------
# multi-GPU: independent replicas (no data-path collective); helpers shared with the CPU tests
# ---------------------------------------------------------------------------------------------
def rank_prompt_range(n_prompts: int, rank: int, world: int):
    """Prompts [lo, hi) of the job's prompt set that rank `rank` of `world` works on: contiguous
    blocks, groups never split.  Its sequence ids start at lo * G."""
    per, extra = divmod(n_prompts, world)
    lo = rank * per + min(rank, extra)
    return lo, lo + per + (1 if rank < extra else 0)


def max_over_ranks(value: float, device, world: int) -> float:
    """The job's time is the slowest rank's time."""
    if world == 1:
        return float(value)
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_second(tokens_per_rank_step: int, world: int, steps: int, elapsed_ms: float) -> float:
    return world * steps * tokens_per_rank_step / (elapsed_ms / 1e3)


# ---------------------------------------------------------------------------------------------
def run_ours(args):
    from paper_2602_02192_b200 import binding, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    peaks = load_peaks()

    wl = synth.WORKLOADS[args.workload]
    shape, P, G, Lp, T = wl.shape, wl.n_prompts, wl.G, wl.prompt_len, wl.new_tokens
    if args.new_tokens:
        T = args.new_tokens
    if args.prompts:
        P = args.prompts
    if args.prompt_len:
        Lp = args.prompt_len
    swap = args.workload == "8B" and not args.no_swap
    nbuf = 1 if args.workload == "32B" else 2
    half_layers = wl.half_layers if args.half_layers < 0 else min(args.half_layers, shape.n_layers)
    eng = binding.Engine(binding.make_config(shape, P, G, Lp, T, nbuf, top_p=args.top_p, half_layers=half_layers),
                         device=local_rank)
    if args.workload == "32B":
        # 65 GB of weights: the snapshot stays in page-locked host memory so that the device holds it once
        weights = synth.make_weights_pinned(shape, wl.weight_seed, gen_device=dev)
    else:
        weights = synth.make_weights(shape, wl.weight_seed, device=dev)
    eng.echo_load_policy(weights, 0)
    eng.echo_wait_policy()
    w_next = None
    if swap:
        del weights
        torch.cuda.empty_cache()
        w_next = synth.make_weights(shape, wl.weight_seed + 1, device=dev)
        torch.cuda.synchronize()

    # Every rank is an independent replica (groups never split): the job's prompt set is world * P
    # prompts, rank r takes prompts [r * P, (r + 1) * P) of it and numbers its sequences from r * P * G,
    # so the job's tokens do not depend on how many GPUs share it.
    all_prompts = synth.make_prompts(world * P, Lp, shape.vocab, wl.prompt_seed)
    lo_p, hi_p = rank_prompt_range(world * P, rank, world)
    prompts = torch.from_numpy(all_prompts[lo_p:hi_p]).to(dev)
    eng.echo_set_sequence_base(lo_p * G)
    lens = [Lp] * P
    out_tok = torch.empty((P, G, T), dtype=torch.int32, device=dev)
    out_lp = torch.empty((P, G, T), dtype=torch.float32, device=dev)

    def one_rollout(seed):
        return eng.echo_rollout(prompts, lens, G, T, wl.temperature, seed, out_tokens=out_tok, out_logprobs=out_lp)

    for w in range(args.warmup):
        one_rollout(wl.sample_seed + w)
    eng.echo_sync()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: K rollouts, device-resident inputs ---------------------------------
    prof_every = max(1, (T - 1) // 16)
    eng.echo_profile_config(prof_every)
    clocks = ClockSampler(local_rank)
    if rank == 0:
        clocks.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    launches = 0
    versions_seen = []
    ev0.record(eng.stream)
    for k in range(args.steps):
        _, _, ver = one_rollout(wl.sample_seed + 100 + k)
        versions_seen.append(int(ver[0, 0]))
        launches += eng.echo_get_stats()["kernels_launched"]
        if swap and k == 0:
            eng.echo_load_policy(w_next, 1)       # overlaps the decode steps already enqueued
    ev1.record(eng.stream)
    eng.echo_sync()
    barrier()
    elapsed_ms = ev0.elapsed_time(ev1)
    clk = clocks.stop() if rank == 0 else None
    prof_steps, prof_ms = eng.echo_profile_read()
    eng.echo_profile_config(0)
    st_last = eng.echo_get_stats()
    install_ms = st_last["install_ms"]
    elapsed_ms = max_over_ranks(elapsed_ms, dev, world)
    value = job_tokens_per_second(P * G * T, world, args.steps, elapsed_ms)

    # ---- end to end: host buffers, copies inside the timed region -------------------------
    hp = prompts.cpu().pin_memory()
    h2d_bytes = int(hp.numel() * 4)
    ht = torch.empty((P, G, T), dtype=torch.int32).pin_memory()
    hl = torch.empty((P, G, T), dtype=torch.float32).pin_memory()
    barrier()
    t0 = time.perf_counter()
    ver_e2e = eng.echo_rollout_host(hp, lens, G, T, wl.temperature, wl.sample_seed + 999, ht, hl)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, dev, world)
    e2e_value = job_tokens_per_second(P * G * T, world, 1, e2e_s * 1e3)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- outside the timed region (rank 0): where the prefill's time goes, and a read-only peak ----
    prefill = None
    eng.echo_profile_config(-1)
    eng.echo_rollout(prompts, lens, G, min(T, 2), wl.temperature, wl.sample_seed + 7, out_tokens=out_tok[:, :, : min(T, 2)].contiguous(),
                     out_logprobs=out_lp[:, :, : min(T, 2)].contiguous())
    pf_steps, pf_ms = eng.echo_profile_read()
    eng.echo_profile_config(0)
    if len(pf_steps) and int(pf_steps[0]) == 0:
        a, g_, _, tot = (float(x) for x in pf_ms[0])
        prefill = {"ms": round(tot, 1), "projections_ms": round(g_, 1), "attention_ms": round(a, 1),
                   "other_ms": round(tot - a - g_, 1),
                   "note": "kernel-by-kernel launches with events (no early start between kernels)"}
    read_gbs = None
    try:
        del hp
        read_gbs = binding.echo_probe_read_bandwidth(2 << 30, 10, device=dev)
    except Exception as e:                      # not enough free memory for the probe buffer
        read_gbs = None

    # ---- roofline of the dominant kernel (decode attention), from the sampled steps ---------
    attn_launches = len(prof_steps) * shape.n_layers
    roof = None
    if attn_launches:
        alg = sum(attention_bytes(shape, P, G, Lp, int(j)) for j in prof_steps) * shape.n_layers
        dur_s = float(prof_ms[:, 0].sum()) / 1e3
        achieved = alg / dur_s / 1e9
        tot = float(prof_ms[:, 3].sum())
        # DRAM bytes per launch: ncu counters of the current kernels on small cases of the same
        # per-CTA work (profiles/attn_decode_kernels_small_cases.md: prefix + suffix launch, DRAM bytes
        # read + written against their algorithmic bytes), scaled to this workload's launches by
        # their algorithmic bytes: the traffic is the KV stream and grows with it.
        traffic = None
        if wl.shape.head_dim == 128:
            small_merge = shape.n_q_heads // shape.n_kv_heads * shape.head_dim <= 512   # resident kernel's limit
            traffic = sum(ATTN_DRAM_PER_ALG_BYTE["resident" if small_merge and int(j) < LONG_SUFFIX_STEP else "waves"] *
                          attention_bytes(shape, P, G, Lp, int(j)) for j in prof_steps) * shape.n_layers / attn_launches
        roof = {"bound": "hbm", "kernel": "decode attention (paged GQA)", "achieved": round(achieved, 1),
                "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
                "frac": round(achieved / peaks["hbm_gbs"], 4),
                "peak_read_only": round(read_gbs, 1) if read_gbs else None,
                "peak_read_only_note": "this library's read-only streaming probe (2 GiB, 16-byte loads, nothing "
                                       "written); the driver's peak is a copy, which also writes",
                "frac_of_read_only_peak": round(achieved / read_gbs, 4) if read_gbs else None,
                "traffic": round(traffic) if traffic else None, "traffic_unit": "bytes per launch (ncu, scaled)",
                "launches_timed": attn_launches,
                "avg_launch_us": round(dur_s / attn_launches * 1e6, 2),
                "sampled_steps": [int(j) for j in prof_steps],
                "share_of_step": {"attention": round(float(prof_ms[:, 0].sum()) / tot, 4),
                                  "projections": round(float(prof_ms[:, 1].sum()) / tot, 4),
                                  "sampler": round(float(prof_ms[:, 2].sum()) / tot, 4)},
                "step_ms": [round(float(x), 3) for x in prof_ms[:, 3]],
                "attn_ms": [round(float(x), 3) for x in prof_ms[:, 0]],
                "gemm_ms": [round(float(x), 3) for x in prof_ms[:, 1]]}
    t_meas = rollout_roofline_seconds(shape, P, G, Lp, T, peaks["hbm_gbs"], peaks["bf16_tflops_sustained"])
    t_nom = rollout_roofline_seconds(shape, P, G, Lp, T, 8000.0, 2250.0)
    per_rollout_s = elapsed_ms / 1e3 / args.steps

    cpu = None
    if not args.no_cpu_baseline:
        cpu = cpu_baseline_sample(eng, shape, w_next if swap else weights, prompts, wl, dev)

    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(elapsed_ms / args.steps, 2), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if half_layers == 0 else f"bf16 (f16 operands in layers 0-{half_layers - 1})",
        "data": "synthetic",
        "config": {"workload": f"{wl.name}-shape decoder: L{shape.n_layers} d{shape.d_model} "
                               f"{shape.n_q_heads}q/{shape.n_kv_heads}kv hd{shape.head_dim} F{shape.d_ff} "
                               f"V{shape.vocab}; {P} prompts x G={G}, prompt {Lp}, {T} new tokens, T=1.0",
                   "top_p": args.top_p, "half_layers": half_layers,
                   "policy_swap": "one echo_load_policy of a re-seeded weight set during timed step 0" if swap
                   else "none", "versions_served": versions_seen, "e2e_version": int(ver_e2e[0, 0]),
                   "install_ms": round(install_ms, 1),
                   "last_rollout_prefill_ms": round(st_last["prefill_ms"], 1), "prefill_breakdown": prefill,
                   "last_rollout_decode_ms_per_step": round(st_last["decode_ms"] / max(1, T - 1), 3),
                   "l2": "inputs larger than L2 (weights + KV >> 126 MB)", "parallelism": f"replicas x{world}"},
        "clocks": clk,
        # time x median SM clock: compares runs on GPUs that settle at different clocks under the power cap
        "sm_gigacycles_per_step": (round(elapsed_ms / args.steps * clk["sm_mhz"] / 1e6, 3)
                                   if clk and clk.get("sm_mhz") else None),
        "e2e": {"value": round(e2e_value, 1), "unit": UNIT, "h2d_bytes_per_step": h2d_bytes,
                "d2h_bytes_per_step": int(ht.numel() * 4 + hl.numel() * 4)},
        "gpu_launches": int(launches),
        "roofline": roof,
        "rollout_roofline": {"frac_of_measured": round(t_meas / per_rollout_s, 4),
                             "frac_of_nominal_8TBs_2250TF": round(t_nom / per_rollout_s, 4),
                             "roofline_s_measured": round(t_meas, 3), "roofline_s_nominal": round(t_nom, 3)},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    eng.close()
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------
def _oracle_dims(shape):
    from oracle import decoder
    return decoder.ModelDims(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                             shape.d_ff, shape.vocab, shape.rms_eps, shape.rope_theta)


class _StreamedWeights:
    """Feeds the oracle one layer at a time from bf16 tensors (exact widening to fp64)."""

    def __init__(self, weights, cache=False):
        self.w = weights
        self.cache = {} if cache else None
        self._wide = lambda t: t.detach().to("cpu").to(torch.float64).numpy()
        self.embed = _EmbedRows(weights["embed"], self._wide)
        self.lm_head = self._wide(weights["lm_head"])
        self.final_norm = self._wide(weights["final_norm"])

    def layer(self, l):
        if self.cache is not None and l in self.cache:
            return self.cache[l]
        lw = {k: self._wide(self.w[k][l]) for k in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down",
                                                    "attn_norm", "mlp_norm")}
        if self.cache is not None:
            self.cache[l] = lw
        return lw


class _EmbedRows:
    def __init__(self, t, wide):
        self.t, self.wide = t, wide

    def __getitem__(self, ids):
        idx = torch.as_tensor(np.asarray(ids), device=self.t.device, dtype=torch.long)
        return self.wide(self.t[idx])


def _oracle_sample_pass(shape, sw, prompt_ids, given, temperature, seed, s):
    from oracle import decoder
    return decoder.score_forced(_oracle_dims(shape), sw, prompt_ids, given, temperature, seed, s,
                                layer_provider=sw.layer)


SAMPLE_PROMPT = 64        # the 8B-shape slice the oracle finishes in tens of seconds
SAMPLE_NEW = 4


def _time_gpu(eng, prompts, lens, G, T, temperature, seed):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    eng.echo_rollout(prompts, lens, G, T, temperature, seed)            # warm-up of this shape of call
    eng.echo_sync()
    e0.record(eng.stream)
    tok, lp, _ = eng.echo_rollout(prompts, lens, G, T, temperature, seed)
    e1.record(eng.stream)
    eng.echo_sync()
    st = eng.echo_get_stats()
    return e0.elapsed_time(e1) / 1e3, st, tok


def cpu_baseline_sample(eng, shape, weights, prompts, wl, dev):
    """The oracle as it stands, timed on this machine's host cores beside the GPU on the SAME inputs:
    (i) the tiny workload in full, KV-cached decoding (mode A); (ii) a slice of this workload."""
    from oracle import decoder
    from paper_2602_02192_b200 import binding, synth
    cores = os.cpu_count() or 1
    # ---- (i) tiny, whole workload, mode A ---------------------------------------------------
    tw = synth.WORKLOADS["tiny"]
    ts = tw.shape
    w_t = synth.make_weights(ts, tw.weight_seed)
    t_prompts = synth.make_prompts(tw.n_prompts, tw.prompt_len, ts.vocab, tw.prompt_seed)
    t_lens = [tw.prompt_len] * tw.n_prompts
    w_o = decoder.Weights(synth.weights_to_bits(w_t))
    t0 = time.perf_counter()
    decoder.rollout_cached(_oracle_dims(ts), w_o, t_prompts, t_lens, tw.G, tw.new_tokens, tw.temperature,
                           tw.sample_seed)
    t_cpu = time.perf_counter() - t0
    n_tiny = tw.n_prompts * tw.G * tw.new_tokens
    teng = binding.Engine(binding.make_config(ts, tw.n_prompts, tw.G, tw.prompt_len, tw.new_tokens, 1),
                          device=torch.device(dev).index or 0)
    teng.echo_load_policy({k: ([t.to(dev) for t in v] if isinstance(v, list) else v.to(dev)) for k, v in w_t.items()}, 1)
    t_gpu, _, _ = _time_gpu(teng, torch.from_numpy(t_prompts).to(dev), t_lens, tw.G, tw.new_tokens, tw.temperature,
                            tw.sample_seed)
    teng.close()
    tiny = {"oracle_tokens_per_s": round(n_tiny / t_cpu, 2), "oracle_s": round(t_cpu, 2),
            "gpu_tokens_per_s": round(n_tiny / t_gpu, 1), "gpu_s": round(t_gpu, 5),
            "sample": f"tiny workload in full ({tw.n_prompts} prompts x G={tw.G}, prompt {tw.prompt_len}, "
                      f"{tw.new_tokens} new tokens), oracle mode A (KV-cached, token by token)"}
    # ---- (ii) a slice of this workload: 1 prompt x G = 1, first SAMPLE_PROMPT prompt tokens, SAMPLE_NEW new tokens
    Lp_s = min(SAMPLE_PROMPT, prompts.shape[1])
    sl_prompts = prompts[:1].clone()
    t_gpu, st, tok = _time_gpu(eng, sl_prompts, [Lp_s], 1, SAMPLE_NEW, wl.temperature, wl.sample_seed)
    given = tok[0, 0].cpu().numpy()
    prompt_ids = sl_prompts[0, :Lp_s].cpu().numpy()
    t0 = time.perf_counter()
    sw = _StreamedWeights(weights)
    t_w = time.perf_counter() - t0
    _oracle_sample_pass(shape, sw, prompt_ids, given, wl.temperature, wl.sample_seed, 0)
    dt = time.perf_counter() - t0
    return {"value": round(SAMPLE_NEW / dt, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
            "seconds": round(dt, 2),
            "sample": f"slice of the {wl.name}-shape workload: 1 prompt x G=1, first {Lp_s} prompt tokens, "
                      f"{SAMPLE_NEW} new tokens, scored teacher-forced along the GPU's tokens in one causal "
                      f"pass (mode C, fp64 numpy), all {shape.n_layers} layers streamed from the bf16 weights "
                      f"(widening included).  A larger slice in KV-cached mode (1 prompt x G=8, prompt 512, 4 tokens, "
                      f"token by token) is beyond a numpy oracle: it re-reads 8 bytes per parameter per token "
                      f"({8 * shape.n_params() / 1e9:.0f} GB at this shape).",
            "gpu_same_input": {"tokens_per_s": round(SAMPLE_NEW / t_gpu, 1), "seconds": round(t_gpu, 5),
                               "prefill_ms": round(st["prefill_ms"], 3), "decode_ms": round(st["decode_ms"], 3)},
            "tiny": tiny}


def run_reference(args):
    """The CPU oracle timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2602_02192_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    shape = wl.shape
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    weights = synth.make_weights(shape, wl.weight_seed, device=dev)
    # the fp64 copy of every layer is kept between steps only where host memory holds it (8 bytes per
    # parameter, on top of the bf16 tensors when those live on the host too); otherwise each step
    # widens the layers again, and the sample description says so
    fp64_bytes = 8 * shape.n_params() + (2 * shape.n_params() if dev == "cpu" else 0)
    try:
        import psutil
        keep = psutil.virtual_memory().available > 1.25 * fp64_bytes
    except Exception:
        keep = False
    sw = _StreamedWeights(weights, cache=keep)
    prompts = synth.make_prompts(wl.n_prompts, wl.prompt_len, shape.vocab, wl.prompt_seed)
    rng = np.random.default_rng(0)
    given = rng.integers(0, shape.vocab, size=SAMPLE_NEW)
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        _oracle_sample_pass(shape, sw, prompts[0, :SAMPLE_PROMPT], given, wl.temperature, wl.sample_seed, 0)
        dt = time.perf_counter() - t0
        if it >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = SAMPLE_NEW * len(times) / total
    cores = os.cpu_count() or 1
    sample = (f"per step: 1 sequence of the {wl.name}-shape workload, first {SAMPLE_PROMPT} prompt tokens + "
              f"{SAMPLE_NEW} tokens scored teacher-forced in one causal pass (fp64 numpy); weights widened "
              + ("to fp64 once before timing" if keep else "to fp64 layer by layer inside every step"))
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(total / len(times) * 1e3, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": f"{wl.name}-shape decoder; bounded sample of {wl.n_prompts} prompts x "
                                   f"G={wl.G}, prompt {wl.prompt_len}, {wl.new_tokens} new tokens"},
            "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_variable_length(args):
    """Diagnostic (--variable-length): responses of uniformly random length in [1, T] (the paper's
    responses average about half the maximum length), produced by teacher-forcing given tokens that
    hold the end token at each sequence's length.  Compares one rollout with the end-of-sequence rule
    (ended sequences are no longer attended) with the same rollout without it.  One JSON line."""
    from paper_2602_02192_b200 import binding, synth
    wl = synth.WORKLOADS[args.workload]
    shape, P, G, Lp = wl.shape, wl.n_prompts, wl.G, wl.prompt_len
    T = args.new_tokens or wl.new_tokens
    weights = synth.make_weights(shape, wl.weight_seed, device="cuda")
    prompts = torch.from_numpy(synth.make_prompts(P, Lp, shape.vocab, wl.prompt_seed)).cuda()
    rng = np.random.default_rng(7)
    eos = shape.vocab - 1
    given = rng.integers(0, eos, size=(P, G, T)).astype(np.int32)
    lengths = rng.integers(1, T + 1, size=(P, G))
    for p in range(P):
        for g in range(G):
            given[p, g, lengths[p, g] - 1:] = eos
    forced = torch.from_numpy(given).cuda()
    out = {}
    for name, eos_id in (("with_rule", eos), ("without_rule", -1)):
        eng = binding.Engine(binding.make_config(shape, P, G, Lp, T, 1, eos_id=eos_id))
        eng.echo_load_policy(weights, 1)
        eng.echo_wait_policy()
        times = []
        for it in range(2):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(eng.stream)
            eng.echo_rollout(prompts, [Lp] * P, G, T, wl.temperature, wl.sample_seed, forced=forced)
            e1.record(eng.stream)
            eng.echo_sync()
            times.append(e0.elapsed_time(e1))
        st = eng.echo_get_stats()
        out[name] = {"ms": round(times[-1], 1), "decode_ms_per_step": round(st["decode_ms"] / max(1, T - 1), 3)}
        eng.close()
        del eng
        torch.cuda.empty_cache()
    useful = int(lengths.sum())
    # A queue of 3 P prompts through the same P group slots: three echo_rollout calls one after the other
    # (each waits for its longest sequence) against one echo_rollout_queue call (a slot is refilled as soon
    # as the host has seen all of its samples ended).
    Q = max(2, args.queue_factor) * P
    q_prompts = torch.from_numpy(synth.make_prompts(Q, Lp, shape.vocab, wl.prompt_seed + 1)).cuda()
    q_given = rng.integers(0, eos, size=(Q, G, T)).astype(np.int32)
    q_len = rng.integers(1, T + 1, size=(Q, G))
    for p in range(Q):
        for g in range(G):
            q_given[p, g, q_len[p, g] - 1:] = eos
    q_forced = torch.from_numpy(q_given).cuda()
    eng = binding.Engine(binding.make_config(shape, P, G, Lp, T, 1, eos_id=eos))
    eng.echo_load_policy(weights, 1)
    eng.echo_wait_policy()
    eng.echo_rollout(prompts, [Lp] * P, G, min(T, 64), wl.temperature, wl.sample_seed)          # warm-up
    eng.echo_sync()
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    e0.record(eng.stream)
    for k in range(Q // P):
        eng.echo_rollout(q_prompts[k * P:(k + 1) * P], [Lp] * P, G, T, wl.temperature, wl.sample_seed,
                         forced=q_forced[k * P:(k + 1) * P])
    e1.record(eng.stream)
    eng.echo_sync()
    tok_q, lp_q, _ = eng.echo_rollout_queue(q_prompts, [Lp] * Q, G, T, wl.temperature, wl.sample_seed, forced=q_forced)
    e2.record(eng.stream)
    eng.echo_sync()
    q_steps = eng.echo_get_stats()["decode_steps"]
    q_useful = int(q_len.sum())
    waves_ms, queue_ms = e0.elapsed_time(e1), e1.elapsed_time(e2)
    base_pages = eng.echo_get_stats()["n_pages"]
    eng.close()
    del eng
    torch.cuda.empty_cache()
    # The same queue with 3 P group slots over the SAME page pool (what P groups need at full length) and
    # at most P*G live sequences: a sample's pages return to the pool when it has ended, so the rows that
    # ended sequences leave are taken by further groups instead of waiting for the slowest sample.
    Z = 16
    pool = P * (-(-Lp // Z)) + P * G * max(-(-(b + T - 1) // Z) for b in range(min(Z, Lp + 1)))
    eng = binding.Engine(binding.make_config(shape, min(Q, 3 * P), G, Lp, T, 1, eos_id=eos, kv_pages=pool,
                                             queue_max_live=P * G))
    eng.echo_load_policy(weights, 1)
    eng.echo_wait_policy()
    eng.echo_rollout_queue(q_prompts[:P], [Lp] * P, G, min(T, 64), wl.temperature, wl.sample_seed)    # warm-up
    eng.echo_sync()
    e3, e4 = (torch.cuda.Event(enable_timing=True) for _ in range(2))
    e3.record(eng.stream)
    tok_o, lp_o, _ = eng.echo_rollout_queue(q_prompts, [Lp] * Q, G, T, wl.temperature, wl.sample_seed, forced=q_forced)
    e4.record(eng.stream)
    eng.echo_sync()
    o_stats = eng.echo_get_stats()
    over_ms = e3.elapsed_time(e4)
    eng.close()
    del eng
    torch.cuda.empty_cache()
    # Optimistic paging on the same pool: pages window by window, up to 2 P G live sequences in 4 P slots,
    # groups evicted and generated again when the pool cannot cover the next window.
    eng = binding.Engine(binding.make_config(shape, min(Q, 4 * P), G, Lp, T, 1, eos_id=eos, kv_pages=pool,
                                             queue_max_live=2 * P * G, queue_optimistic=3))
    eng.echo_load_policy(weights, 1)
    eng.echo_wait_policy()
    eng.echo_rollout_queue(q_prompts[:P], [Lp] * P, G, min(T, 64), wl.temperature, wl.sample_seed)    # warm-up
    eng.echo_sync()
    e5, e6 = (torch.cuda.Event(enable_timing=True) for _ in range(2))
    e5.record(eng.stream)
    tok_p, lp_p, _ = eng.echo_rollout_queue(q_prompts, [Lp] * Q, G, T, wl.temperature, wl.sample_seed, forced=q_forced)
    e6.record(eng.stream)
    eng.echo_sync()
    p_stats = eng.echo_get_stats()
    opt_ms = e5.elapsed_time(e6)
    opt_same = float((tok_p == tok_q).float().mean())
    opt_gap = float((lp_p - lp_q).abs().mean())
    same = float((tok_o == tok_q).float().mean())
    gap = (lp_o - lp_q).abs().flatten()
    lp_gap = float(gap.mean())
    lp_gap_q = float(torch.quantile(gap[:: max(1, gap.numel() // 1000000)].float(), 0.999))
    eng.close()
    queue = {"prompts": Q, "slots": P, "useful_tokens": q_useful,
             "calls_of_P_prompts": {"ms": round(waves_ms, 1), "decode_steps": (Q // P) * (T - 1),
                             "useful_tokens_per_s": round(q_useful / waves_ms * 1e3, 1)},
             "one_queue_call": {"ms": round(queue_ms, 1), "decode_steps": int(q_steps), "kv_pages": int(base_pages),
                                "useful_tokens_per_s": round(q_useful / queue_ms * 1e3, 1)},
             "one_queue_call_3x_slots_same_pool": {
                 "ms": round(over_ms, 1), "decode_steps": int(o_stats["decode_steps"]), "slots": min(Q, 3 * P), "kv_pages": int(pool),
                 "kv_pages_peak": int(o_stats["n_pages"]), "max_live_sequences": P * G,
                 "useful_tokens_per_s": round(q_useful / over_ms * 1e3, 1),
                 "tokens_equal_to_the_P_slot_queue": round(same, 4), "mean_logprob_gap": round(lp_gap, 5),
                 "q999_logprob_gap": round(lp_gap_q, 4)},
             "one_queue_call_optimistic_pages_same_pool": {
                 "ms": round(opt_ms, 1), "decode_steps": int(p_stats["decode_steps"]), "slots": min(Q, 4 * P),
                 "kv_pages": int(pool), "kv_pages_peak": int(p_stats["n_pages"]), "max_live_sequences": 2 * P * G,
                 "groups_evicted": int(p_stats["queue_evictions"]),
                 "useful_tokens_per_s": round(q_useful / opt_ms * 1e3, 1),
                 "tokens_equal_to_the_P_slot_queue": round(opt_same, 4), "mean_logprob_gap": round(opt_gap, 5)}}
    print(json.dumps({"diagnostic": "variable-length responses, teacher-forced", "workload": wl.name, "max_new_tokens": T,
                      "queue": queue,
                      "mean_length": round(float(lengths.mean()), 1), "useful_tokens": useful,
                      "with_rule": out["with_rule"], "without_rule": out["without_rule"],
                      "useful_tokens_per_s_with_rule": round(useful / out["with_rule"]["ms"] * 1e3, 1),
                      "useful_tokens_per_s_without_rule": round(useful / out["without_rule"]["ms"] * 1e3, 1)}))


def run_projections(args):
    """Diagnostic (--projections): every projection shape of one decode step of the workload, alone,
    with rotating weight sets larger than L2, through echo_gemm_bf16 (SM-pair kernel, block-tiled
    weights, fused epilogue) and, as context, through torch.matmul (cuBLAS, bf16 output, no epilogue).
    One JSON line per shape."""
    from paper_2602_02192_b200 import binding, synth
    lib = binding.lib
    wl = synth.WORKLOADS[args.workload]
    sh = wl.shape
    M = wl.n_prompts * wl.G
    dev = torch.device("cuda:0")
    nws = int(lib.echo_gemm_workspace_bytes(M))
    ws = torch.empty(nws, dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    qkv = (sh.n_q_heads + 2 * sh.n_kv_heads) * sh.head_dim
    # qkv: the engine's q/k/v projection adds into a buffer that the kernel consuming it leaves zeroed
    # (epilogue 1 here); a stand-alone store (epilogue 0) would time a memset of the output as well
    shapes = [("qkv", qkv, sh.d_model, 1), ("o", sh.d_model, sh.n_q_heads * sh.head_dim, 1),
              ("gate_up_swiglu", sh.d_ff, sh.d_model, 2), ("down", sh.d_model, sh.d_ff, 1),
              ("lm_head", sh.vocab, sh.d_model, 0)]

    def timed(fn, iters):
        for i in range(max(4, iters // 4)):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / iters

    for name, N, K, epi in shapes:
        rows_w = 2 * N if epi == 2 else N
        nbuf = 2 if rows_w * K * 2 > 400e6 else int(400e6 // (rows_w * K * 2)) + 2
        Ws = [torch.empty(rows_w, K, device=dev, dtype=torch.bfloat16).normal_(0, 0.02) for _ in range(nbuf)]
        X = torch.empty(M, K, device=dev, dtype=torch.bfloat16).normal_()
        Y = torch.zeros(M, N, device=dev, dtype=torch.bfloat16 if epi == 2 else torch.float32)
        Yb = torch.empty(M, rows_w, device=dev, dtype=torch.bfloat16)
        # timing only: the same buffers stand in for block-tiled storage (identical size for these shapes)
        impl = 1300 if M > 64 else 1000

        def ours(i):
            rc = lib.echo_gemm_bf16(X.data_ptr(), Ws[i % nbuf].data_ptr(), Y.data_ptr(), M, N, K, epi, impl,
                                    ws.data_ptr(), nws, st)
            assert rc == 0, rc

        def cublas(i):
            torch.matmul(X, Ws[i % nbuf].t(), out=Yb)

        t_ours, t_lib = timed(ours, 10 * nbuf), timed(cublas, 10 * nbuf)
        flops = 2.0 * M * rows_w * K
        print(json.dumps({"projection": name, "rows": M, "features": rows_w, "k": K, "epilogue": epi,
                          "us": round(t_ours, 2), "weights_gbs": round(rows_w * K * 2 / t_ours / 1e3, 1),
                          "tflops": round(flops / t_ours / 1e6, 1), "cublas_us": round(t_lib, 2),
                          "cublas_tflops": round(flops / t_lib / 1e6, 1)}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8B", choices=["tiny", "0.6B", "4B", "8B", "32B"])
    ap.add_argument("--new-tokens", type=int, default=0, help="override T (diagnostic runs only)")
    ap.add_argument("--prompts", type=int, default=0, help="override the number of prompts (diagnostic runs only)")
    ap.add_argument("--prompt-len", type=int, default=0, help="override the prompt length (diagnostic runs only)")
    ap.add_argument("--no-swap", action="store_true")
    ap.add_argument("--top-p", type=float, default=1.0,
                    help="nucleus sampling (the paper samples with 0.95); 1.0 = the benchmark's untruncated sampling")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--half-layers", type=int, default=-1,
                    help="leading layers with IEEE-half operands; default: the workload's setting")
    ap.add_argument("--queue-factor", type=int, default=3,
                    help="--variable-length: prompts in the queue, as a multiple of the workload's prompt count")
    ap.add_argument("--variable-length", action="store_true",
                    help="diagnostic: random response lengths with and without the end-of-sequence rule, and exit")
    ap.add_argument("--projections", action="store_true",
                    help="diagnostic: time each projection shape alone (with cuBLAS beside it) and exit")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and not (
            args.variable_length or args.projections):
        # one process per GPU: start the ranks (the same command line under the torch launcher)
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        os.execv(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                  f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
                                  "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:])
    if args.variable_length:
        run_variable_length(args)
    elif args.projections:
        run_projections(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
