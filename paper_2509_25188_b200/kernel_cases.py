"""Runs one kernel of the denoising step stand-alone, at a layer's real shapes, and times it.

  python -m paper_2509_25188_b200.kernel_cases gate_up --rows 512 [--iters 20] [--tile-n 0]

Cases (LLaDA-8B layer shapes unless overridden with --d/--ff/--vocab/--heads):
  qkv      C[T,3d]  = A[T,d] Wqkv^T                 bf16 store epilogue
  o        X[T,d]  += A[T,d] Wo^T                   residual epilogue
  gate_up  H[T,F]   = silu(A Wg^T) * (A Wu^T)       SwiGLU epilogue
  down     X[T,d]  += H[T,F] Wd^T                   residual epilogue
  lm_head  pred/conf over V for R = --rows rows     fused confidence head
  attn     bidirectional attention, --rows queries and keys, 32 heads x 128
  train    filter training (Algorithm 1, stage 2): --rows samples of 32 confidences, --iters epochs per call
  step     whole denoising steps of a --layers deep model of these widths (batch 1, --rows / 2 prompt
           tokens + --rows / 2 masks, block 32): the small, self-ending case for profiling the
           memory-bound kernels (RMSNorm, RoPE/scatter, embedding, final norm, decision)

Each iteration uses a different weight buffer out of a ring larger than L2 (126 MB), so that the
weights come from HBM as they do inside a step.  Prints one JSON line with the mean device time
(CUDA events on the launching stream) and the achieved TFLOP/s and GB/s.  Used for tuning and as
the small, self-ending case for profiler captures.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as b


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["qkv", "o", "gate_up", "down", "lm_head", "attn", "step", "train"])
    ap.add_argument("--rows", type=int, default=512)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--tile-n", type=int, default=0)
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--ff", type=int, default=12288)
    ap.add_argument("--vocab", type=int, default=126464)
    ap.add_argument("--heads", type=int, default=32)
    ap.add_argument("--layers", type=int, default=2, help="step: number of layers")
    ap.add_argument("--kv-cache", type=int, default=0, help="step: 0 = every step runs all --rows positions; 1 / 2 = prefix / dual "
                    "cache: the timed steps are in-block steps of the first block (at most 31 of them in all)")
    ap.add_argument("--chain", type=int, default=0, help="step: 0 = one launch per projection, 1 = chained launches (one persistent "
                    "launch per layer), 2 = the chained form's tiling in single launches")
    ap.add_argument("--trace", action="store_true", help="step with --chain 1: also print the phases' time stamps of the last step "
                    "(per launch and phase: when the slowest CTA opened it, had its last accumulator ready, finished it)")
    ap.add_argument("--impl", type=int, default=0, help="attn: 0 = tcgen05 kernel, 1 = mma.sync kernel")
    ap.add_argument("--sustain", type=float, default=0.0, help="also run the launches back to back for this many seconds while the "
                    "SM clock is sampled (NVML, read-only): time per launch, median MHz and their product in the power-capped state")
    ap.add_argument("--ring", type=int, default=0, help="number of weight buffers to rotate through (0 = enough to exceed L2)")
    a = ap.parse_args()
    dev = "cuda:0"
    torch.manual_seed(0)
    T, d, F, V, H = a.rows, a.d, a.ff, a.vocab, a.heads
    dh = d // H

    def rnd(r, c, std=0.02):
        return (torch.randn(r, c, device=dev) * std).to(torch.bfloat16)

    def ring(r, c, min_bytes=400e6):
        n = a.ring if a.ring > 0 else max(2, int(min_bytes // (r * c * 2)) + 1)
        return [rnd(r, c) for _ in range(n)]

    if a.case == "step":
        from . import workloads as wl
        shape = wl.ModelShape(n_layers=a.layers, d_model=d, n_heads=H, head_dim=dh, d_ff=F, vocab=V, rms_eps=1e-5,
                              rope_theta=500000.0, mask_id=V - 1, eot_id=V - 2, dtype="bf16")
        ones = torch.ones(d, device=dev)
        w = {"tok_emb": rnd(V, d), "lm_head": rnd(V, d),
             "final_norm": torch.full((d,), wl.spread_gain(shape), device=dev),
             "layers": [{"wqkv": rnd(3 * d, d), "wo": rnd(d, d), "w_gate": rnd(F, d), "w_up": rnd(F, d),
                         "w_down": rnd(d, F), "norm1": ones, "norm2": ones} for _ in range(a.layers)]}
        dec = b.Decoder(shape, w, wl.make_filter(32, 0.96, seed=0), block_len=32, max_batch=1, max_seq=T,
                        kv_cache=a.kv_cache, use_filter=a.kv_cache == 0)
        prompts = torch.from_numpy(wl.make_prompts(1, T // 2, shape, seed=1)).to(dev)
        dec.set_chain(a.chain)
        if a.kv_cache:
            # one commit per step: the first block has 31 steps that read the store
            assert a.warmup + 2 * a.iters <= 31, "at most 31 in-block steps"
            dec.state_reset_device(prompts, T - T // 2)
            dec.denoise_step(outputs=False)

        def run(i):
            if not a.kv_cache:
                dec.state_reset_device(prompts, T - T // 2)
            dec.denoise_step(outputs=False)
        per_layer = 2.0 * T * (4 * d * d + 3 * d * F) + 4.0 * T * T * d
        flops, byts = a.layers * per_layer + 2.0 * 32 * d * V, 2.0 * (a.layers * (4 * d * d + 3 * d * F) + V * d)
    elif a.case == "train":
        import numpy as np
        from . import workloads as wl
        rng = np.random.default_rng(0)
        c_s = torch.from_numpy(rng.uniform(0.0, 1.0, size=(T, 32)).astype(np.float32)).to(dev)
        y_s = (c_s + 0.15 * torch.randn_like(c_s) > 0.6).to(torch.uint8)
        f0 = wl.make_filter(32, 0.96, seed=0)
        epochs = 10
        run = lambda i: b.filter_train(f0, c_s, y_s, epochs)
        flops, byts = epochs * 10.0 * T * 32 * 32, epochs * 5.0 * T * 32
    elif a.case == "qkv":
        A, W = rnd(T, d, 1.0), ring(3 * d, d)
        Cc = torch.empty(T, 3 * d, dtype=torch.bfloat16, device=dev)
        run = lambda i: b._check(b.lib.l2pd_gemm_bf16(b._stream(), A.data_ptr(), W[i % len(W)].data_ptr(),
                                                      Cc.data_ptr(), T, 3 * d, d, a.tile_n, 0))
        flops, byts = 2.0 * T * d * 3 * d, 2.0 * (3 * d * d + T * d + T * 3 * d)
    elif a.case == "o":
        A, W, X = rnd(T, d, 1.0), ring(d, d), torch.zeros(T, d, device=dev)
        run = lambda i: b._check(b.lib.l2pd_gemm_bf16_residual(b._stream(), A.data_ptr(), W[i % len(W)].data_ptr(),
                                                               X.data_ptr(), T, d, d, a.tile_n, 0))
        flops, byts = 2.0 * T * d * d, 2.0 * (d * d + T * d) + 8.0 * T * d
    elif a.case == "gate_up":
        A, Wg, Wu = rnd(T, d, 1.0), ring(F, d, 200e6), ring(F, d, 200e6)
        Hh = torch.empty(T, F, dtype=torch.bfloat16, device=dev)
        run = lambda i: b._check(b.lib.l2pd_gemm_bf16_swiglu(b._stream(), A.data_ptr(), Wg[i % len(Wg)].data_ptr(),
                                                             Wu[i % len(Wu)].data_ptr(), Hh.data_ptr(), T, F, d,
                                                             a.tile_n, 0))
        flops, byts = 2.0 * T * d * 2 * F, 2.0 * (2 * F * d + T * d + T * F)
    elif a.case == "down":
        A, W, X = rnd(T, F, 1.0), ring(d, F), torch.zeros(T, d, device=dev)
        run = lambda i: b._check(b.lib.l2pd_gemm_bf16_residual(b._stream(), A.data_ptr(), W[i % len(W)].data_ptr(),
                                                               X.data_ptr(), T, d, F, a.tile_n, 0))
        flops, byts = 2.0 * T * d * F, 2.0 * (d * F + T * F) + 8.0 * T * d
    elif a.case == "lm_head":
        A, W = rnd(T, d, 1.0), ring(V, d, 1.1e9)
        scratch = torch.empty(b.lib.l2pd_lm_head_scratch_elems(T, V), device=dev)
        pred = torch.empty(T, dtype=torch.int32, device=dev)
        conf = torch.empty(T, device=dev)

        def run(i):
            b._check(b.lib.l2pd_lm_head_bf16(b._stream(), A.data_ptr(), W[i % len(W)].data_ptr(), None, T, V, d,
                                             scratch.data_ptr(), pred.data_ptr(), conf.data_ptr(), None, 0))
        flops, byts = 2.0 * T * d * V, 2.0 * (V * d + T * d)
    else:
        q, k, v = rnd(T, d, 1.0), rnd(T, d, 1.0), rnd(T, d, 1.0)
        out = torch.empty(T, d, dtype=torch.bfloat16, device=dev)
        run = lambda i: b._check(b.lib.l2pd_attention_bf16(b._stream(), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                                           out.data_ptr(), T, T, H, dh, d, d, d, a.impl, 0))
        flops, byts = 4.0 * T * T * d, 2.0 * 4 * T * d

    for i in range(a.warmup):
        run(i)
    torch.cuda.synchronize()
    # a device wait that ran out leaves its code in the library's status word: the checked call below reports it
    probe = torch.zeros(16, 64, dtype=torch.bfloat16, device=dev)
    b.gemm_bf16(probe, torch.zeros(64, 64, dtype=torch.bfloat16, device=dev))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tot = 0.0
    for i in range(a.iters):
        e0.record()
        run(i)
        e1.record()
        torch.cuda.synchronize()
        tot += e0.elapsed_time(e1)
    ms = tot / a.iters
    # the same launches back to back (no host synchronisation in between)
    e0.record()
    for i in range(a.iters):
        run(i)
    e1.record()
    torch.cuda.synchronize()
    ms_b2b = e0.elapsed_time(e1) / a.iters
    sustained = None
    if a.sustain > 0:
        import statistics
        import threading
        import time
        import pynvml
        pynvml.nvmlInit()
        h = pynvml.nvmlDeviceGetHandleByIndex(torch.cuda.current_device())
        n = max(a.iters, int(a.sustain * 1e3 / ms_b2b))
        mhz, stop = [], threading.Event()

        def sample():
            while not stop.is_set():
                mhz.append(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
                time.sleep(0.02)
        th = threading.Thread(target=sample)
        th.start()
        e0.record()
        for i in range(n):
            run(i)
        e1.record()
        torch.cuda.synchronize()
        stop.set()
        th.join()
        us = e0.elapsed_time(e1) / n * 1e3
        med = statistics.median(mhz[len(mhz) // 3:]) if len(mhz) >= 3 else None   # the clock settles within the first third
        sustained = {"launches": n, "us": us, "sm_mhz_median": med, "kcycles": us * med / 1e3 if med else None,
                     "tflops": flops / us / 1e6}
    if a.case == "step" and a.trace and a.chain == 1:
        import numpy as np
        dec.chain_trace_enable(True)
        run(0)
        tr = dec.chain_trace()
        dec.chain_trace_enable(False)
        if tr is not None:
            tr = tr.astype(np.int64)
            names = ["O", "norm2", "gate_up", "down", "norm1", "QKV"]
            for launch in range(tr.shape[0]):
                n = 1 if launch == 0 else (6 if launch < tr.shape[0] - 1 else 4)
                t = tr[launch, :n]
                t0, prev = t[0, 0].min(), t[0, 0].min()
                row = []
                for ph in range(n):
                    op, r1, r2, fin = t[ph]
                    busy = r2 > op
                    row.append({"phase": names[ph] if launch else "QKV", "us": round((fin.max() - prev) / 1e3, 2),
                                "main_loop_us_median": round(float(np.median((r1 - op)[busy])) / 1e3, 2) if busy.any() else 0.0,
                                "drain_us_median": round(float(np.median((fin - r2)[busy])) / 1e3, 2) if busy.any() else 0.0})
                    prev = fin.max()
                print(json.dumps({"launch": launch, "total_us": round((t[n - 1, 3].max() - t0) / 1e3, 2), "phases": row}))
    print(json.dumps({"case": a.case, "rows": T, "tile_n": a.tile_n, "ms": ms, "ms_back_to_back": ms_b2b, "tflops_b2b": flops / ms_b2b / 1e9, "tflops": flops / ms / 1e9,
                      "gbs": byts / ms / 1e6, "flops": flops, "bytes": byts, "sustained": sustained}))


if __name__ == "__main__":
    main()
