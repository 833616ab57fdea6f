#!/usr/bin/env python
"""Benchmark of the Learn2PD denoising step and decode on B200.

  python bench.py --gpus N --steps K --warmup W            (this implementation)
  python bench.py --impl reference --steps K --warmup W    (the CPU oracle, timed as it stands)

Timed step (N = 1 and every replica at N > 1): one denoising step of the LLaDA-8B-shaped model — batch 1, 256
prompt tokens + 256 masked positions, block 32 — i.e. the state set-up of Algorithm 2 followed by M(X), the
confidence head, the filter, the threshold and EoTP.  A "step" of the timed loop is exactly that, repeated K times
on the same seeded prompt; `ms_per_step` is its time.  `value` (generated tokens per second) is measured on the full
Learn2PD decode of the same model and prompt shape (256 + 256, EoT logit biased so that EoTP fires): tokens up to
and including [EoT] over the decode's device time, summed over ranks.
With --gpus N > 1 and no launcher environment the script starts its N ranks itself (one per GPU, NCCL).
Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2509_25188_b200 import workloads as wl  # noqa: E402

WORKLOAD = "C1"
SHAPE = wl.LLADA_8B
DEC = wl.DECODES[WORKLOAD]
METRIC, UNIT = "generated_tokens_per_s", "tokens/s"
EOT_BIAS = 14.0          # the seeded constant added to the [EoT] logit in the decode workloads
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes of one gate/up launch at 512 rows, from the ncu capture summarised under profiles/ (null when absent)
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "gate_up_T512_dram_traffic.txt")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def measured_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, or None."""
    try:
        for line in open(TRAFFIC_FILE):
            if line.startswith("bytes_per_launch"):
                return float(line.split("=")[1].split("#")[0])
    except OSError:
        pass
    return None


def step_work(shape, T, Lk, R, kv_read_bytes=0.0):
    """Algorithmic FLOPs and bytes of one denoising step over T rows, Lk keys per query, R LM-head rows."""
    d, F, V, NL = shape.d_model, shape.d_ff, shape.vocab, shape.n_layers
    hd = shape.n_heads * shape.head_dim
    gemm = 2.0 * T * NL * (d * 3 * hd + hd * d + 3 * d * F)
    attn = 4.0 * NL * hd * T * Lk
    head = 2.0 * R * d * V
    w_bytes = 2.0 * (NL * (d * 3 * hd + hd * d + 3 * d * F) + V * d)
    act_bytes = 44.0 * T * d * NL
    return {"flops": gemm + attn + head, "weight_bytes": w_bytes, "act_bytes": act_bytes, "kv_bytes": kv_read_bytes}


def roofline_ms(work, pk):
    """The slower of FLOPs at the bf16 peak and bytes at the HBM peak, for the burst and the sustained bf16 figure."""
    t_bytes = (work["weight_bytes"] + work["act_bytes"] + work.get("kv_bytes", 0.0)) / (pk["hbm_gbs"] * 1e9)
    t_burst = max(work["flops"] / (pk["bf16_tflops"] * 1e12), t_bytes)
    t_sust = max(work["flops"] / (pk["bf16_tflops_sustained"] * 1e12), t_bytes)
    bound = "tensor" if work["flops"] / (pk["bf16_tflops"] * 1e12) >= t_bytes else "hbm"
    return 1e3 * t_burst, 1e3 * t_sust, 1e3 * t_bytes, bound


def config_dict():
    return {"workload": "%s: one denoising step, LLaDA-8B-shaped model (32 layers, d 4096, 32 heads x 128, "
                        "SwiGLU 12288, vocab 126464), batch 1, prompt %d + %d masked, block %d, filter + EoTP "
                        "(ms_per_step); value = generated tokens/s of the full decode of the same shape (C2)"
                        % (WORKLOAD, DEC.prompt_len, DEC.gen_len, DEC.block_len),
            "tokens_per_step_rows": DEC.prompt_len + DEC.gen_len, "block_len": DEC.block_len, "tau": DEC.tau,
            "eot_bias": EOT_BIAS,
            "l2": "inputs larger than L2: every step streams 15 GB of weights",
            "weights": "N(0, 0.02^2) bf16, drawn on the device with torch's generator, seed 0",
            "parallelism": "replicas"}


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference): whole steps of the full-depth model, measured

class OracleStep:
    """The oracle as it stands, one call = one whole denoising step of the 32-layer model (embedding, every layer over
    the sequence's rows, LM head on the block's rows, confidence head, decision).  fresh(): the C1 step (state set-up,
    then the first step); next(): the following step of the same decode (the C2 workload, EoT logit biased)."""

    def __init__(self, eot_bias=None):
        from oracle import l2pd_oracle as orc
        self.orc = orc
        t0 = time.perf_counter()
        w = wl.make_weights(SHAPE, seed=0, final_norm_gain=wl.spread_gain(SHAPE), threads=os.cpu_count() or 8)
        self.setup_s = time.perf_counter() - t0
        self.model = orc.Model(n_layers=SHAPE.n_layers, d_model=SHAPE.d_model, n_heads=SHAPE.n_heads, head_dim=SHAPE.head_dim,
                               d_ff=SHAPE.d_ff, vocab=SHAPE.vocab, rms_eps=SHAPE.rms_eps, rope_theta=SHAPE.rope_theta,
                               mask_id=SHAPE.mask_id, eot_id=SHAPE.eot_id, weights=w,
                               lm_head_bias=None if eot_bias is None else wl.make_eot_bias(SHAPE, eot_bias))
        self.filt = wl.make_filter(DEC.block_len, DEC.tau, seed=0)
        self.prompt = wl.make_prompts(1, DEC.prompt_len, SHAPE, seed=1)[0]
        self.cfg = orc.DecodeConfig(block_len=DEC.block_len, tau=DEC.tau)
        self.st = None

    def fresh(self):
        self.st = self.orc.init_state(self.model, self.prompt, DEC.gen_len)
        return self.next()

    def next(self):
        """Returns (seconds, positions the step committed)."""
        t0 = time.perf_counter()
        rec = self.orc.denoise_step(self.model, self.filt, self.st, self.cfg)
        return time.perf_counter() - t0, int(rec.unmask.sum())


def oracle_cores():
    import threadpoolctl
    return max(i["num_threads"] for i in threadpoolctl.threadpool_info() or [{"num_threads": os.cpu_count()}])


def run_reference(args):
    """The oracle on a bounded sample of the decode workload `value` is quoted on: the first steps of the C2 decode of
    sequence 0 (whole 32-layer steps, measured one by one), as many of the K asked as fit the time budget or until the
    first block is fully unmasked; value = positions those steps committed / their time."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleStep(eot_bias=EOT_BIAS)
    cores = oracle_cores()
    budget_s = 150.0                     # a step is ~30 s on 16 cores
    times, toks = [], 0
    t, n = smp.fresh()
    times.append(t)
    toks += n
    while (len(times) < args.steps and not smp.st.done and smp.st.cur_block == 0
           and sum(times) + 1.2 * max(times) < budget_s):
        t, n = smp.next()
        times.append(t)
        toks += n
    total = sum(times)
    value = toks / total
    sample = ("the first %d denoising steps of the C2 decode of sequence 0 (of %d asked), each a whole step of the 32-layer model "
              "measured directly (~%.0f s each; no warm-up step: a step is tens of seconds; weights drawn in %.0f s beforehand); "
              "they committed %d of the first block's %d positions; value = those tokens / their time"
              % (len(times), args.steps, total / len(times), smp.setup_s, toks, DEC.block_len))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(times), "steps_requested": args.steps, "warmup": 0, "warmup_requested": args.warmup,
            "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(), "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU leg

def device_weights(shape, device, seed=0):
    """Random-init weights drawn on the device (same distribution as workloads.make_weights)."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    d, F, V = shape.d_model, shape.d_ff, shape.vocab
    hd = shape.n_heads * shape.head_dim

    def mat(r, c):
        return (torch.randn(r, c, generator=g, device=device, dtype=torch.float32) * 0.02).to(torch.bfloat16)

    ones = torch.ones(d, device=device, dtype=torch.float32)
    layers = []
    for _ in range(shape.n_layers):
        layers.append({"wqkv": mat(3 * hd, d), "wo": mat(d, hd), "w_gate": mat(F, d), "w_up": mat(F, d),
                       "w_down": mat(d, F), "norm1": ones, "norm2": ones})
    return {"tok_emb": mat(V, d), "lm_head": mat(V, d),
            "final_norm": torch.full((d,), wl.spread_gain(shape), device=device, dtype=torch.float32), "layers": layers}


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            pass
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.count(",") >= 8]
        os.unlink(self.f.name)
        if not rows:
            return out
        sm = [float(r[1]) for r in rows]
        out["sm_mhz"] = statistics.median(sm)
        out["sm_max_mhz"] = float(rows[0][2])
        out["power_w_max"] = max(float(r[3]) for r in rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        out["reasons"] = [n for i, n in enumerate(names) if any("Active" == r[5 + i].strip() for r in rows)]
        out["samples"] = len(rows)
        return out


def traced_decode(dec, d_prompts, G):
    """The decode as state set-up + step loop, with each step's device time and row count (for per-step rooflines)."""
    dec.state_reset_device(d_prompts, G)
    rec = []
    while dec.num_active > 0:
        h = dec.denoise_step_host()
        rec.append((dec.last_step_ms, dec.last_step_rows, h["l_eff"].copy(), h["done"].copy()))
    return rec


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2509_25188_b200 import binding, replicas

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    multi = replicas.launcher_env_present()      # started by a launcher (any world size): the process-group path runs
    if multi:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    pk, pk_src = peaks()

    w = device_weights(SHAPE, dev)
    filt = wl.make_filter(DEC.block_len, DEC.tau, seed=0)
    B, P, G, s = DEC.batch, DEC.prompt_len, DEC.gen_len, DEC.block_len
    dec = binding.Decoder(SHAPE, w, filt, block_len=s, tau=DEC.tau, max_batch=B, max_seq=P + G, device=local)
    prompts = wl.make_prompts(B, P, SHAPE, seed=1 + rank)
    h_prompts = torch.from_numpy(prompts).pin_memory()
    d_prompts = h_prompts.to(dev)

    def barrier():
        if multi:
            dist.barrier()
        torch.cuda.synchronize()

    def one_resident():
        dec.state_reset_device(d_prompts, G)
        return dec.denoise_step_host()

    warm = max(args.warmup, 3)
    for _ in range(warm):
        one_resident()

    # ---- timed region 1: K denoising steps, inputs resident in HBM
    sampler = ClockSampler(local) if rank == 0 else None
    dec.profile_enable(["gemm_gate_up"])
    launches0 = dec.launch_count
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    step_ms = []
    for _ in range(args.steps):
        one_resident()
        step_ms.append(dec.last_step_ms)      # the library's own events around this step (the call has synchronised)
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    launches = dec.launch_count - launches0
    prof = dec.profile_read()
    dec.profile_enable([])

    # ---- timed region 2: the same steps end to end — host prompt in, host results out, every step
    dev_in = torch.empty_like(d_prompts)
    o_conf = torch.empty(B, s, device=dev)
    o_pred = torch.empty(B, s, dtype=torch.int32, device=dev)
    o_un = torch.empty(B, s, dtype=torch.uint8, device=dev)
    h_conf, h_pred, h_un = (torch.empty_like(t, device="cpu").pin_memory() for t in (o_conf, o_pred, o_un))
    barrier()
    ev0.record()
    for _ in range(args.steps):
        dev_in.copy_(h_prompts, non_blocking=True)
        dec.state_reset_device(dev_in, G)
        dec.denoise_step_into(o_conf, o_pred, o_un)
        h_conf.copy_(o_conf, non_blocking=True)
        h_pred.copy_(o_pred, non_blocking=True)
        h_un.copy_(o_un, non_blocking=True)
        torch.cuda.current_stream().synchronize()
    ev1.record()
    barrier()
    ms_e2e_step = ev0.elapsed_time(ev1)

    # ---- timed region 3: full Learn2PD decodes (C2).  Two per rank, handed out from a queue shared by the ranks
    # (a rank that is done takes the next one), gathered over the process group at the end.
    bias = wl.make_eot_bias(SHAPE, EOT_BIAS)
    dec2 = binding.Decoder(SHAPE, w, filt, block_len=s, tau=DEC.tau, max_batch=B, max_seq=P + G, device=local, lm_head_bias=bias)
    n_dec = 2 * world
    dec_prompts = wl.make_prompts(n_dec, P, SHAPE, seed=1)            # sequence 0 = the prompt of the timed step
    h_dec_prompts = torch.from_numpy(dec_prompts).pin_memory()
    d_one = torch.empty(1, P, dtype=torch.int32, device=dev)
    d_out = torch.empty(1, G, dtype=torch.int32, device=dev)
    h_out = torch.empty(1, G, dtype=torch.int32).pin_memory()
    d_one.copy_(h_dec_prompts[0:1])
    dec2.decode_device(d_one, G, d_out)                                # warm-up at the decode's shapes
    if multi:
        store = dist.distributed_c10d._get_default_store()
    idx, toks, lens, stps = [], [], [], []
    dec_ms = dec_ms_e2e = 0.0
    barrier()
    t_wall0 = time.perf_counter()
    chunks = replicas.claim_chunks(store, n_dec) if multi else iter(range(n_dec))
    for i in chunks:
        # end to end: the prompt comes from pinned host memory and the response goes back to it, inside the timed region
        ev0.record()
        d_one.copy_(h_dec_prompts[i:i + 1], non_blocking=True)
        ev_in = torch.cuda.Event(enable_timing=True)
        ev_in.record()
        out_len, seq_steps, total_steps = dec2.decode_device(d_one, G, d_out)
        ev_out = torch.cuda.Event(enable_timing=True)
        ev_out.record()
        h_out.copy_(d_out, non_blocking=True)
        ev1.record()
        torch.cuda.synchronize()
        dec_ms += ev_in.elapsed_time(ev_out)
        dec_ms_e2e += ev0.elapsed_time(ev1)
        idx.append(i)
        toks.append(h_out.numpy().copy())
        lens.append(int(out_len[0]))
        stps.append(int(seq_steps[0]))
    barrier()
    wall_ms = 1e3 * (time.perf_counter() - t_wall0)
    toks_np = np.concatenate(toks) if toks else np.zeros((0, G), np.int32)
    if multi:
        all_toks, all_len, all_steps = replicas.gather_indexed(idx, toks_np, np.array(lens), np.array(stps), n_dec, G, device=dev)
        dec_ms, (_,) = replicas.reduce_timing(dec_ms, [0.0], device=dev)
        dec_ms_e2e, (_,) = replicas.reduce_timing(dec_ms_e2e, [0.0], device=dev)
        ms, (launches,) = replicas.reduce_timing(ms, [launches], device=dev)
        ms_e2e_step, (_,) = replicas.reduce_timing(ms_e2e_step, [0.0], device=dev)
        launches = int(launches)
    else:
        all_toks, all_len, all_steps = toks_np, np.array(lens), np.array(stps)
    clocks = sampler.stop() if sampler else None
    gen_tokens = float(np.sum(all_len))
    value = gen_tokens / (dec_ms * 1e-3)                 # all ranks' tokens over the slowest rank's decode time
    value_e2e = gen_tokens / (dec_ms_e2e * 1e-3)

    line = None
    if rank == 0:
        T, R = B * (P + G), B * s
        work = step_work(SHAPE, T, P + G, R)
        t_burst, t_sust, t_bytes, bound = roofline_ms(work, pk)
        ms_step = ms / args.steps
        gu_ms, gu_n = prof.get("gemm_gate_up", (0.0, 0))
        gu_flops = 2.0 * T * SHAPE.d_model * 2 * SHAPE.d_ff
        achieved = gu_flops / (gu_ms / gu_n * 1e-3) / 1e12 if gu_n else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": ms_step, "ms_per_step_median": statistics.median(step_ms), "ms_per_step_min": min(step_ms),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": config_dict(), "clocks": clocks,
            "e2e": {"value": value_e2e, "unit": UNIT, "ms_per_step": ms_e2e_step / args.steps,
                    "what": "decodes with the prompt copied from pinned host memory and the response copied back inside the timed "
                            "region (value); ms_per_step: the timed step with its prompt copied in and conf / pred / unmask copied out",
                    "h2d_bytes_per_step": int(h_prompts.numel() * 4),
                    "d2h_bytes_per_step": int(h_conf.numel() * 4 + h_pred.numel() * 4 + h_un.numel() + 6 * 4 * B + 4)},
            "gpu_launches": int(launches),
            "roofline": {"kernel": "gemm_tcgen05_pair_kernel<EPI_SWIGLU> (gate/up projection + SwiGLU)", "bound": "tensor",
                         "achieved": achieved, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": (achieved / pk["bf16_tflops"]) if achieved else None,
                         "peak_source": pk_src + " (burst bf16)",
                         "frac_sustained": (achieved / pk["bf16_tflops_sustained"]) if achieved else None,
                         "flops_per_launch": gu_flops, "avg_launch_ms": gu_ms / gu_n if gu_n else None,
                         "traffic": measured_traffic(),
                         "algorithmic_bytes": 2.0 * (2 * SHAPE.d_ff * SHAPE.d_model + T * SHAPE.d_model + T * SHAPE.d_ff)},
            "step_roofline": {"flops": work["flops"], "weight_bytes": work["weight_bytes"], "act_bytes": work["act_bytes"],
                              "bound": bound, "t_bytes_ms": t_bytes, "t_roof_ms": t_burst, "frac": t_burst / ms_step,
                              "t_roof_sustained_ms": t_sust, "frac_sustained": t_sust / ms_step,
                              "mcycles_per_step": (ms_step * clocks["sm_mhz"] / 1e3) if clocks and clocks.get("sm_mhz") else None,
                              "note": "frac: against the burst bf16 figure (the target's denominator); frac_sustained: against the "
                                      "seconds-long figure under the power cap; mcycles_per_step: ms_per_step x the median SM clock "
                                      "sampled during the timed region (what the step costs in SM cycles, whatever clock the power "
                                      "cap allowed)",
                              "peaks": pk, "peak_source": pk_src},
            "decode": {"workload": "C2: full Learn2PD decode, prompt %d + generation %d, block %d, filter + EoTP, EoT logit biased "
                                   "by the constant %.1f; %d sequences (2 per rank, taken from a shared queue)" % (P, G, s, EOT_BIAS, n_dec),
                       "sequences": n_dec, "out_len": [int(v) for v in all_len], "steps_per_sequence": float(np.mean(all_steps)),
                       "steps_one_token_per_step": G, "device_ms_slowest_rank": dec_ms, "wall_ms": wall_ms,
                       "generated_tokens_per_s": value},
        }

    # ---- untimed, rank 0: per-kernel breakdown of the step; per-step rooflines of a decode; the other configurations
    if rank == 0:
        dec.profile_enable(binding.KINDS)
        for _ in range(3):
            one_resident()
        line["breakdown"] = {k: {"ms_per_step": round(t_ms / 3, 4), "launches_per_step": n // 3}
                             for k, (t_ms, n) in dec.profile_read().items()}
        dec.profile_enable([])

        # the decode of sequence 0 step by step: each step's roofline from its actual row count (T = L_eff keys = rows here)
        d_one.copy_(h_dec_prompts[0:1])
        rec = traced_decode(dec2, d_one, G)
        t_meas = sum(r[0] for r in rec)
        roofs = [roofline_ms(step_work(SHAPE, rows, rows, s), pk) for (_, rows, _, _) in rec]
        line["decode"]["per_step"] = {
            "steps": len(rec), "rows_first_last": [rec[0][1], rec[-1][1]], "ms_total": t_meas,
            "roofline_ms_total": sum(r[0] for r in roofs), "frac_time_weighted": sum(r[0] for r in roofs) / t_meas,
            "frac_time_weighted_sustained": sum(r[1] for r in roofs) / t_meas,
            "note": "sum over the decode's steps of each step's roofline (from its own T = L_q = L_k and R = 32) / sum of their device times"}
    dec2.close()
    dec.close()

    if rank == 0 and not args.no_other_configs:
        line["other_configs"] = other_configs(binding, torch, w, filt, pk, dev, local)
    if rank == 0 and args.extra_workloads:
        line["extra_workloads"] = extra_workloads(binding, torch, w, filt, dev, local)

    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            del w
            torch.cuda.empty_cache()
            smp = OracleStep()
            t_step, n_tok = smp.fresh()
            line["cpu_baseline"] = {
                "value": n_tok / t_step, "unit": UNIT, "cores": oracle_cores(), "kind": "oracle", "ms_per_step": 1e3 * t_step,
                "sample": "one whole denoising step of the C1 workload (32 layers, 512 rows, LM head on 32 rows, decision) measured "
                          "directly: %.1f s; tokens = the %d positions that step committed; compare ms_per_step with ms_per_step"
                          % (t_step, n_tok)}
        print(json.dumps(line))
    if multi:
        dist.barrier()
        dist.destroy_process_group()


def other_configs(binding, torch, w, filt, pk, dev, local):
    """First / cached steps of the batched configurations and the dual cache's in-block step, each with its roofline
    (burst and sustained bf16 figure).  Bounded: a few steps per configuration."""
    s = DEC.block_len
    out = {}

    def frac(work, t_ms):
        t_burst, t_sust, _, bound = roofline_ms(work, pk)
        return {"ms": t_ms, "roofline_ms": t_burst, "frac": t_burst / t_ms, "roofline_sustained_ms": t_sust,
                "frac_sustained": t_sust / t_ms, "bound": bound}

    for name in ("C3", "C4"):
        dsh = wl.DECODES[name]
        Bx, Px, Gx = dsh.batch, dsh.prompt_len, dsh.gen_len
        decx = binding.Decoder(SHAPE, w, filt, block_len=s, tau=dsh.tau, max_batch=Bx, max_seq=Px + Gx, device=local,
                               kv_cache=dsh.kv_cache)
        px = torch.from_numpy(wl.make_prompts(Bx, Px, SHAPE, seed=100)).to(dev)

        def first_step():
            decx.state_reset_device(px, Gx)
            decx.denoise_step_host()
            return decx.last_step_ms
        first_step()
        t_first = statistics.median(first_step() for _ in range(3))
        Tx = Bx * (Px + Gx)
        rec = {"rows": Tx, "first_step": frac(step_work(SHAPE, Tx, Px + Gx, Bx * s), t_first)}
        if dsh.kv_cache:
            decx.state_reset_device(px, Gx)
            decx.denoise_step_host()
            times = []
            for _ in range(3):
                if decx.num_active == 0:
                    break
                decx.denoise_step_host()
                times.append((decx.last_step_ms, decx.last_step_rows))
            if times:
                t_c, rows_c = times[-1]
                kv = 2.0 * 2 * SHAPE.n_layers * Bx * Px * SHAPE.n_heads * SHAPE.head_dim     # stored K and V of the prefix, read once
                rec["cached_step"] = dict(rows=rows_c, **frac(step_work(SHAPE, rows_c, Px + Gx, Bx * s, kv), t_c))
        out[name] = rec
        decx.close()
    # dual cache (Section 4.3): in-block steps run the block's s rows per sequence against the stored keys and values
    for name, dsh in (("C2_dual_cache", wl.DECODES["C2"]), ("C4_dual_cache", wl.DECODES["C4"])):
        Bx, Px, Gx = dsh.batch, dsh.prompt_len, dsh.gen_len
        decx = binding.Decoder(SHAPE, w, None, block_len=s, tau=dsh.tau, max_batch=Bx, max_seq=Px + Gx, device=local,
                               kv_cache=2, use_filter=False)      # one commit per step: s - 1 stored-key steps per block
        px = torch.from_numpy(wl.make_prompts(Bx, Px, SHAPE, seed=100)).to(dev)
        decx.state_reset_device(px, Gx)
        decx.denoise_step_host()
        t_first = decx.last_step_ms
        for _ in range(3):
            decx.denoise_step_host()
        times = []
        for _ in range(10):
            decx.denoise_step_host()
            times.append(decx.last_step_ms)
        rows = decx.last_step_rows
        kv = 2.0 * 2 * SHAPE.n_layers * Bx * (Px + Gx) * SHAPE.n_heads * SHAPE.head_dim
        out[name] = dict(rows=rows, first_step_ms=t_first,
                         in_block_step=frac(step_work(SHAPE, rows, Px + Gx, Bx * s, kv), statistics.median(times)))
        decx.close()
    # the C2 decode of the headline (filter + EoTP, same prompts and EoT bias) with the key/value caches of Section 4.3
    dsh = wl.DECODES["C2"]
    prompts = torch.from_numpy(wl.make_prompts(2, dsh.prompt_len, SHAPE, seed=1)).to(dev)
    d_out = torch.empty(1, dsh.gen_len, dtype=torch.int32, device=dev)
    bias = wl.make_eot_bias(SHAPE, EOT_BIAS)
    for mode, key in ((1, "C2_decode_prefix_cache"), (2, "C2_decode_dual_cache")):
        decx = binding.Decoder(SHAPE, w, filt, block_len=s, tau=dsh.tau, max_batch=1, max_seq=dsh.prompt_len + dsh.gen_len,
                               device=local, kv_cache=mode, lm_head_bias=bias)
        decx.decode_device(prompts[0:1], dsh.gen_len, d_out)      # warm-up
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        lens, steps = [], []
        ev0.record()
        for i in range(2):
            ln, st, _ = decx.decode_device(prompts[i:i + 1], dsh.gen_len, d_out)
            lens.append(int(ln[0])); steps.append(int(st[0]))
        ev1.record()
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1)
        out[key] = {"sequences": 2, "out_len": lens, "steps": steps, "ms": ms, "generated_tokens_per_s": sum(lens) / (ms * 1e-3),
                    "note": "the cached steps approximate the keys and values of positions outside the current block, so the "
                            "trajectory (steps, length) differs from the uncached decode's"}
        decx.close()
    return out


def extra_workloads(binding, torch, w, filt, dev, local):
    """Long generation with and without EoTP, the threshold / policy sweep on the C2 decode and filter training at the
    paper's scale (Sections 4.3-4.4, Algorithm 1): behaviour of the loop on the synthetic model, outside the contract's
    numbers.  --extra-workloads."""
    B, P, G, s = DEC.batch, DEC.prompt_len, DEC.gen_len, DEC.block_len
    d_prompts = torch.from_numpy(wl.make_prompts(B, P, SHAPE, seed=1)).to(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    extra = {}
    # long generation (the setting of Section 4.3's EoTP study: generation length 1024, block 32): one sequence, the
    # EoT logit biased so that the answer ends early; the same decode with and without EoTP
    Pl, Gl, bias_l = 1024, 1024, 14.0
    pl_ = torch.from_numpy(wl.make_prompts(1, Pl, SHAPE, seed=7)).to(dev)
    out_l = torch.empty(1, Gl, dtype=torch.int32, device=dev)
    rec = {"prompt_len": Pl, "gen_len": Gl, "eot_bias": bias_l}
    for tag, eotp in (("eotp", True), ("no_eotp", False)):
        decl = binding.Decoder(SHAPE, w, filt, block_len=s, tau=DEC.tau, max_batch=1, max_seq=Pl + Gl, device=local,
                               use_eotp=eotp, lm_head_bias=wl.make_eot_bias(SHAPE, bias_l))
        decl.state_reset_device(pl_, Gl)
        decl.denoise_step_host()                       # warm-up at this shape
        ev0.record()
        ol, st_l, tot_l = decl.decode_device(pl_, Gl, out_l)
        ev1.record()
        torch.cuda.synchronize()
        first_eot = (out_l[0] == SHAPE.eot_id).nonzero()
        rec[tag] = {"ms": ev0.elapsed_time(ev1), "steps": int(tot_l), "out_len": int(ol[0]),
                    "first_eot": int(first_eot[0]) if len(first_eot) else -1}
        decl.close()
    rec["speedup_from_eotp"] = rec["no_eotp"]["ms"] / rec["eotp"]["ms"]
    extra["long_generation"] = rec

    # threshold sweep (Section 4.4 studies tau = 0.9 ... 0.99) and the comparison policies on the C2 decode: steps and
    # generated tokens per second of one sequence with the same synthetic model, filter and EoT bias
    sweep = {}
    d_out2 = torch.empty(B, G, dtype=torch.int32, device=dev)
    for tag, kw, rule in [("tau_0.90", {"tau": 0.90}, None), ("tau_0.96", {"tau": 0.96}, None), ("tau_0.99", {"tau": 0.99}, None),
                          ("confidence_0.9", {"tau": DEC.tau}, ("confidence", 0.9)),
                          ("one_token_per_step", {"tau": DEC.tau}, ("confidence", 1.0))]:
        decs = binding.Decoder(SHAPE, w, filt, block_len=s, max_batch=B, max_seq=P + G, device=local,
                               lm_head_bias=wl.make_eot_bias(SHAPE, 14.0), **kw)
        if rule:
            decs.set_unmask_rule(rule[0], conf_threshold=rule[1])
        decs.state_reset_device(d_prompts, G)
        decs.denoise_step_host()
        ev0.record()
        ol, st_s, tot_s = decs.decode_device(d_prompts, G, d_out2)
        ev1.record()
        torch.cuda.synchronize()
        ms_s = ev0.elapsed_time(ev1)
        sweep[tag] = {"steps": int(tot_s), "out_len": int(ol[0]), "ms": ms_s,
                      "generated_tokens_per_s": float(np.sum(ol)) / (ms_s * 1e-3)}
        decs.close()
    base_steps = sweep["one_token_per_step"]["steps"]
    for v in sweep.values():
        v["steps_vs_one_token_per_step"] = base_steps / max(v["steps"], 1)
    extra["policy_sweep_C2"] = sweep

    # filter training at the paper's scale (Section 4.1: 2,640 prompts, 5,000 epochs, lr 0.001): synthetic samples,
    # one per decoding step of a 32-step-per-prompt EGP run; the whole of stage 2 on the device
    n_samp = 2640 * 32
    rng = np.random.default_rng(0)
    c_s = rng.uniform(0.0, 1.0, size=(n_samp, s)).astype(np.float32)
    y_s = (c_s + 0.15 * rng.normal(size=(n_samp, s)) > 0.6).astype(np.uint8)
    tc_s, ty_s = torch.from_numpy(c_s).to(dev), torch.from_numpy(y_s).to(dev)
    binding.filter_train(filt, tc_s, ty_s, 20)
    ev0.record()
    _, tr_losses = binding.filter_train(filt, tc_s, ty_s, 5000)
    ev1.record()
    torch.cuda.synchronize()
    ms_tr = ev0.elapsed_time(ev1)
    fl_epoch = 10.0 * n_samp * s * s        # two products forward, three backward, 2 flops per multiply-add
    extra["filter_training"] = {"samples": n_samp, "block_len": s, "epochs": 5000, "batch": "full", "ms": ms_tr,
                                "us_per_epoch": 1e3 * ms_tr / 5000, "gflops": fl_epoch * 5000 / (ms_tr * 1e-3) / 1e9,
                                "loss_first": float(tr_losses[0]), "loss_last": float(tr_losses[-1])}

    return extra


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--extra-workloads", action="store_true",
                    help="also run the long-generation pair (with / without EoTP), the threshold and policy sweep on the C2 decode "
                         "and filter training at the paper's scale; reported under extra_workloads, outside the contract's numbers")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the steps of the batched configurations (C3, C4) and of the dual cache")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    from paper_2509_25188_b200 import replicas
    if args.gpus > 1 and not replicas.launcher_env_present():
        # no launcher started us: start the N ranks ourselves, one per GPU
        sys.exit(replicas.spawn_local_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    run_ours(args)


if __name__ == "__main__":
    main()
