#!/usr/bin/env python
"""Benchmark of the MREM reconstruction step.

A step = one pass of the whole hot path (weight quantization, teacher forward, student
forward, loss, straight-through backward, AdamW) over one calibration batch of one module.
Default workload: a BERT-large module of 6 layers, W4A8, batch 32 x seq 128, bf16 storage,
drawn from a 1024-sequence seeded synthetic calibration set that lives in HBM.

    python bench.py --gpus 1 --steps 20 --warmup 3
    python bench.py --impl reference            # the CPU oracle, as it stands, on the host cores

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
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "recon-step tokens/sec (fwd+bwd) per BERT-large W4A8 module"
UNIT = "tokens/s"
INT8_OVER_BF16 = 2.0        # nominal dense int8 : bf16 tensor throughput on this part


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "20"], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- CPU oracle leg

def oracle_sample(wl, n_steps=1, warmup=0, batch=None):
    """Times the oracle, as it stands, on ONE layer of the module with the full batch
    (teacher forward, student forward, loss, backward, AdamW) and extrapolates to the
    module's layer count.  Returns (tokens/s, threads used, description, seconds per sample)."""
    from oracle import mrem_oracle as O
    from paper_2109_15082_b200 import synth
    batch = batch or wl.batch
    one = synth.shrink(wl, n_layers=1, batch=batch)
    params = synth.teacher_params(one, 0)
    x = synth.hidden_states(one, batch, 0)
    vl = synth.valid_lengths(one, batch, 0)
    desc = O.ModuleDesc(1, wl.hidden, wl.n_heads, wl.ffn, wl.w_bits, wl.a_bits, wl.w_grid, act_dtype=wl.act_dtype)
    student = [{k: v.copy() for k, v in params[0].items()}]
    ws = O.init_weight_steps(desc, student, wl.w_step_rule)
    a, off = O.init_act_steps(desc, student, x, vl)
    steps, state = O.make_steps(ws, a, off), {}
    times = []
    for i in range(warmup + n_steps):
        t0 = time.perf_counter()
        O.recon_step(desc, params, student, steps, state, x, x, vl, lr=wl.lr)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    sec = sum(times) / len(times)
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    tokens = batch * wl.seq
    desc_txt = (f"1 of {wl.n_layers} layers, batch {batch}x{wl.seq} of {wl.batch}x{wl.seq}, teacher fwd + student fwd + loss + "
                f"backward + AdamW in float64 numpy; tokens/s extrapolated as tokens / ({wl.n_layers} x t_layer)")
    return tokens / (wl.n_layers * sec), threads, desc_txt, sec


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # each step is a bounded sample of the batch, sized so that the whole run stays within a few minutes: one
    # sequence through one layer of the module costs the oracle about 0.2 s on 16 cores
    batch = max(1, min(wl.batch, 700 // max(args.steps + min(args.warmup, 1), 1)))
    val, threads, sample, sec = oracle_sample(wl, n_steps=max(1, args.steps), warmup=min(args.warmup, 1), batch=batch)
    # `value` is the rate of the workload's metric; each timed step really ran `batch` sequences through ONE of the
    # module's layers (`ms_timed_per_step`), and `ms_per_step` scales that to the whole module and batch
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec * wl.n_layers * wl.batch / batch,
            "ms_timed_per_step": 1e3 * sec, "extrapolated": True,
            "extrapolation": {"layers_timed": 1, "layers": wl.n_layers, "sequences_timed": batch, "sequences": wl.batch},
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, wl.calib or wl.batch * 8, 1),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(wl, calib_n, world):
    """The `config` object of the JSON line; both arms print the same keys."""
    return {"workload": wl.name, "layers": wl.n_layers, "hidden": wl.hidden, "heads": wl.n_heads,
            "ffn": wl.ffn, "batch": wl.batch, "seq_len": wl.seq, "bits": f"W{wl.w_bits}A{wl.a_bits}",
            "calibration_sequences": calib_n, "parallelism": "replicas only" if world > 1 else "1 GPU",
            "l2": "inputs larger than L2: calibration set, weights and optimizer state exceed 126 MB",
            "launch": "one CUDA-graph replay per step + 2 gather kernels"}


# ----------------------------------------------------------------------------- GPU leg

def ncu_dram_bytes_per_launch(workload, kernel):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel` from the committed ncu summary of this
    workload (profiles/tc_gemm_dram_<workload>.md, line `traffic_bytes_per_launch <kernel> = <bytes>`), or None when
    there is no such capture.  Returns (bytes, file)."""
    import re
    path = os.path.join(ROOT, "profiles", f"tc_gemm_dram_{workload}.md")
    if not os.path.exists(path):
        return None, None
    m = re.search(r"traffic_bytes_per_launch\s+" + re.escape(kernel) + r"\s*=\s*([0-9.eE+]+)", open(path).read())
    return (float(m.group(1)), os.path.relpath(path, ROOT)) if m else (None, None)


def build_problem(wl, rank, torch, calib_n):
    from paper_2109_15082_b200 import synth
    from paper_2109_15082_b200.session import ReconModule
    m = ReconModule(wl.n_layers, wl.hidden, wl.n_heads, wl.ffn, wl.seq, wl.batch, wl.w_bits, wl.a_bits, wl.w_grid,
                    True, 3, wl.act_dtype)
    m.load_teacher(synth.teacher_params(wl, seed=rank))          # rank = replica seed: independent problems
    m.init_student_from_teacher()
    m.init_weight_steps(wl.w_step_rule)
    calib = torch.empty(calib_n, wl.seq, wl.hidden, dtype=m.tdtype, device=m.device)
    chunk = 64
    for c0 in range(0, calib_n, chunk):
        n = min(chunk, calib_n - c0)
        x = synth.hidden_states(wl, n, seed=rank, tag=f"calib{c0}")
        calib[c0:c0 + n].copy_(torch.from_numpy(x).to(m.device))
    lens = torch.from_numpy(synth.valid_lengths(wl, calib_n, seed=rank)).to(m.device)
    return m, calib, lens


def run_data_parallel(args, wl):
    """--dp: ONE module on all ranks (identical parameters), every step's batch split over the ranks; per layer one
    all-reduce (NCCL, sum) of the gradient bucket before the update (paper_2109_15082_b200/dist.py).  Strong scaling:
    the whole job processes one batch of the workload per step whatever the number of ranks.  Eager call sequence (the
    update has to wait for the all-reduce, so the step is not one captured graph here)."""
    import torch
    import torch.distributed as dist
    from paper_2109_15082_b200 import binding as B
    from paper_2109_15082_b200 import dist as D
    from paper_2109_15082_b200 import synth
    from paper_2109_15082_b200.session import ReconModule
    rank, world, local = D.env_rank()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl")
    W, K = max(3, args.warmup), args.steps
    calib_n = args.calib or wl.calib or wl.batch * 8
    lo, hi = D.shard_bounds(wl.batch, rank, world)
    nb = hi - lo
    if nb < 1:
        raise RuntimeError("--dp needs at least one sequence of the batch per rank")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        m = ReconModule(wl.n_layers, wl.hidden, wl.n_heads, wl.ffn, wl.seq, nb, wl.w_bits, wl.a_bits, wl.w_grid, True, 3, wl.act_dtype)
        m.load_teacher(synth.teacher_params(wl, seed=0))              # the same module on every rank
        m.init_student_from_teacher()
        m.init_weight_steps(wl.w_step_rule)
        calib = torch.empty(calib_n, wl.seq, wl.hidden, dtype=m.tdtype, device=m.device)
        for c0 in range(0, calib_n, 64):
            n = min(64, calib_n - c0)
            calib[c0:c0 + n].copy_(torch.from_numpy(synth.hidden_states(wl, n, seed=0, tag=f"calib{c0}")).to(m.device))
        lens = torch.from_numpy(synth.valid_lengths(wl, calib_n, seed=0)).to(m.device)
        total = W + K
        n_batches = calib_n // wl.batch
        perm = np.concatenate([synth.permutation(0, f"epoch{e}", calib_n)[: n_batches * wl.batch]
                               for e in range((total + n_batches - 1) // n_batches + 1)])
        idx = torch.from_numpy(perm[: total * wl.batch].reshape(total, wl.batch)[:, lo:hi].astype(np.int32).copy()).to(m.device)
        lens_steps = lens[idx.long()].contiguous()
        xbuf = torch.empty(nb, wl.seq, wl.hidden, dtype=m.tdtype, device=m.device)
        row_bytes = wl.seq * wl.hidden * xbuf.element_size()
        dp = D.DataParallelModule(m)

        def step(t):
            B.mrem_gather_rows(calib, idx[t], nb, row_bytes, xbuf, side.cuda_stream)
            return dp.step(xbuf, xbuf, lens_steps[t], nb, wl.batch, wl.seq, opt)

        B.mrem_gather_rows(calib, idx[0], nb, row_bytes, xbuf, side.cuda_stream)
        dp.init_act_steps(xbuf, lens_steps[0], nb, wl.seq)
        opt = B.make_optim(lr=wl.lr, step=0, decay_total_steps=max(wl.steps, total))
        for t in range(W):
            step(t)
        side.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        for t in range(W, W + K):
            loss = step(t)
        e1.record(side)
        side.synchronize()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        clocks = sampler.stop() if rank == 0 else None
        ms = D.max_over_ranks(e0.elapsed_time(e1), m.device)
        loss_last = float(loss[0])
        status = m.poll_status()
        bucket_bytes = sum(int(b.numel()) * 4 for b in dp.buckets)
        m.close()
    if rank == 0:
        tokens = wl.batch * wl.seq
        cfg = workload_config(wl, calib_n, world)
        cfg.update(parallelism=f"dp{world}: batch split over the ranks, one gradient all-reduce per layer",
                   launch="eager call sequence (the update waits for the all-reduce)", sequences_per_rank=nb,
                   allreduce_bytes_per_step=bucket_bytes)
        print(json.dumps({"metric": METRIC, "value": tokens * K / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                          "ms_per_step": ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
                          "dtype": "bf16+int8", "data": "synthetic", "config": cfg, "clocks": clocks, "e2e": None,
                          "gpu_launches": None, "loss_last": loss_last, "device_status": status,
                          "note": "data-parallel mode; with one rank it is the eager call sequence of the step"}))
    if world > 1:
        dist.destroy_process_group()


def time_extras(m, wl, xbuf, lenbuf, stream, torch, B, pk, reps=10):
    """Device times (CUDA events, after 3 warm-up calls) of the entry points beside the module step, on the workload's
    shapes: one step of Eq. 2 per weight matrix of a layer on batch x seq rows, the output-logit term inside
    mrem_recon_loss, and one embedding step (BERT-large tables when the workload is BERT-large)."""
    from paper_2109_15082_b200.embedding import EmbeddingStep

    def timed(fn, n=reps):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream.synchronize()
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        stream.synchronize()
        return e0.elapsed_time(e1) / n

    out = {}
    rows = wl.batch * wl.seq
    opt = B.make_optim(lr=wl.lr, step=0, decay_total_steps=100000)
    x2 = xbuf.reshape(rows, wl.hidden)
    g_in = torch.randn(rows, wl.ffn, device=m.device, dtype=torch.float32).abs().to(m.tdtype)     # FFN2 input: non-negative like a GELU output
    rem = {}
    for name, pid, a, n_out, n_in in (("Wqkv", B.WQKV, x2, 3 * wl.hidden, wl.hidden), ("Wo", B.WO, x2, wl.hidden, wl.hidden),
                                      ("W1", B.W1, x2, wl.ffn, wl.hidden), ("W2", B.W2, g_in, wl.hidden, wl.ffn)):
        ms = timed(lambda: m.rem_step(0, pid, a, opt))
        flop = 4 * 2.0 * rows * n_out * n_in                   # teacher product, integer product, weight gradient, input gradient
        rem[name] = {"ms_per_step": ms, "tflops": flop / (ms * 1e-3) / 1e12}
    out["rem_step"] = {"rows": rows, "per_matrix": rem,
                       "note": "Eq. 2 on one product: two forward products (bf16, int8), loss, two backward products, fused update"}
    # output-logit term: mrem_recon_loss with and without a bound head (3 classes)
    m.quantize_weights()
    m.forward_teacher(xbuf, lenbuf, wl.batch, wl.seq)
    m.forward_student(xbuf, lenbuf, wl.batch, wl.seq)
    plain = timed(lambda: m.recon_loss())
    rng = np.random.default_rng(0)
    H = wl.hidden
    m.bind_head(dict(Wp=rng.normal(0, 1 / np.sqrt(H), (H, H)), bp=np.zeros(H), Wc=rng.normal(0, 1 / np.sqrt(H), (3, H)), bc=np.zeros(3)))
    with_head = timed(lambda: m.recon_loss())
    m.bind_head(None)
    out["logit_term"] = {"recon_loss_ms": plain, "recon_loss_with_head_ms": with_head, "classes": 3}
    # embedding step
    V, P = (30522, 512) if wl.hidden >= 768 else (1000, 64)
    teacher = dict(word=rng.normal(0, 0.05, (V, H)), pos=rng.normal(0, 0.02, (max(P, wl.seq), H)), type=rng.normal(0, 0.02, (2, H)),
                   ln_g=np.ones(H), ln_b=np.zeros(H))
    emb = EmbeddingStep(teacher, 4, rows, wl.act_dtype, stream=stream)
    emb.set_student(None, np.abs(teacher["word"]).max(1) / 7)
    ids = torch.from_numpy((rng.zipf(1.2, (wl.batch, wl.seq)) % V).astype(np.int32)).to(m.device)
    ms = timed(lambda: emb.step(ids, None, opt))
    table_bytes = V * H * (4 + 16 + 12 + 1)                     # gradient cleared; w, g, m, v read; w, m, v, code written
    out["embed_step"] = {"vocab": V, "tokens": rows, "e_bits": 4, "ms_per_step": ms, "table_gbs": table_bytes / (ms * 1e-3) / 1e9,
                         "hbm_peak_gbs": pk["hbm_gbs"], "status": int(emb.status[0]),
                         "note": "whole step; table_gbs counts only the dense pass over the word table (33 B per entry)"}
    # the module step with weight scales recomputed from the weights (w_grid 3: refitted W4 scales; w_grid 2: ternary)
    from paper_2109_15082_b200 import synth as _synth
    from paper_2109_15082_b200.session import ReconModule as _RM
    cf = {}
    for label, grid, bits in (("refit_w4", 3, 4), ("ternary_w2", 2, 2)):
        with torch.cuda.stream(stream):
            mc = _RM(wl.n_layers, wl.hidden, wl.n_heads, wl.ffn, wl.seq, wl.batch, bits, wl.a_bits, grid, True, 3, wl.act_dtype,
                     stream=stream)
            mc.load_teacher(_synth.teacher_params(wl, seed=7))
            mc.init_student_from_teacher()
            mc.init_act_steps(xbuf, lenbuf, wl.batch, wl.seq)
            stream.synchronize()
            B.mrem_graph_capture_step(mc.ctx, xbuf, xbuf, 0.0, lenbuf, wl.batch, wl.seq, mc.t_out, mc.s_out, mc.loss, opt)
            ms = timed(lambda: B.mrem_graph_launch(mc.ctx), n=20)
            cf[label] = {"ms_per_step": ms, "tokens_per_s": rows / (ms * 1e-3), "loss": float(mc.loss[:1].item())}
            mc.close()
    out["closed_form_scales"] = cf
    # the whole sequential sweep of the stated BERT-large configuration: 4 modules of the workload's depth one after the
    # other, 200 steps each over a 1024-sequence calibration set, outputs cached for the next module (wall clock,
    # synchronised at both ends; includes step initialisation, graph capture and the caching passes)
    if wl.name == "large6_w4a8":
        from paper_2109_15082_b200 import synth
        from paper_2109_15082_b200.session import ReconModule
        from paper_2109_15082_b200.sweep import ModuleSweep
        n_mod, steps, n_cal = 4, 200, 1024
        with torch.cuda.stream(stream):
            mods = []
            for k in range(n_mod):
                mk = ReconModule(wl.n_layers, wl.hidden, wl.n_heads, wl.ffn, wl.seq, wl.batch, wl.w_bits, wl.a_bits, wl.w_grid, True, 3,
                                 wl.act_dtype, stream=stream)
                mk.load_teacher(synth.teacher_params(wl, seed=100 + k))
                mk.init_student_from_teacher()
                mods.append(mk)
            calib = torch.randn(n_cal, wl.seq, wl.hidden, device=m.device, dtype=torch.float32).to(m.tdtype)
            lens = torch.randint(32, wl.seq + 1, (n_cal,), device=m.device, dtype=torch.int32)
            sweep = ModuleSweep(mods, calib, lens, wl.batch, lambda k, e: synth.permutation(k, f"sweep{e}", n_cal), wl.w_step_rule)
            stream.synchronize()
            t0 = time.perf_counter()
            for k in range(n_mod):
                sweep.run_module(k, steps, B.make_optim(lr=wl.lr, step=0, decay_total_steps=steps), record_every=50)
                if k + 1 < n_mod:
                    sweep.cache_outputs(k)
            stream.synchronize()
            dt = time.perf_counter() - t0
            out["sweep"] = {"modules": n_mod, "layers_per_module": wl.n_layers, "steps_per_module": steps, "calibration_sequences": n_cal,
                            "seconds": dt, "tokens_per_s": n_mod * steps * rows / dt,
                            "first_and_last_recorded_loss": [[l[0], l[-1]] for l in sweep.losses]}
            for mk in mods:
                mk.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large6_w4a8")
    ap.add_argument("--calib", type=int, default=0, help="calibration sequences (0: the workload's)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--extras", action="store_true", help="also time the per-product step (Eq. 2), the output-logit term and the "
                    "embedding step of the first module, and add them to the JSON line as \"extras\"")
    ap.add_argument("--no-pdl", action="store_true", help="plain stream-ordered launches (no programmatic dependent launch)")
    ap.add_argument("--dp", action="store_true", help="data parallel: one module, each step's batch split over the ranks, gradients "
                    "all-reduced per layer (strong scaling); default is one independent replica per rank")
    ap.add_argument("--repeats", type=int, default=0, help="timed blocks of --steps steps each (0: as many as bring the timed "
                    "region to about 2 s, between 3 and 64); the line reports the median block and the fastest")
    args = ap.parse_args()

    from paper_2109_15082_b200 import synth
    wl = synth.workloads()[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
        return

    if args.dp:
        run_data_parallel(args, wl)
        return

    import torch
    import torch.distributed as dist
    from paper_2109_15082_b200 import binding as B

    from paper_2109_15082_b200 import dist as D
    rank, world, local = D.env_rank()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    if args.no_pdl:
        B.mrem_set_programmatic_launch(0)
    if world > 1:
        dist.init_process_group("nccl")
    W = max(3, args.warmup)
    K = args.steps
    calib_n = args.calib or wl.calib or wl.batch * 8
    tokens = wl.batch * wl.seq
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        m, calib, lens = build_problem(wl, rank, torch, calib_n)
        max_repeats = args.repeats if args.repeats > 0 else 64
        total = W + K * min(max_repeats, 8)                           # batches drawn; later blocks start over at W
        n_batches = calib_n // wl.batch
        perm = np.concatenate([synth.permutation(rank, f"epoch{e}", calib_n)[: n_batches * wl.batch]
                               for e in range((total + n_batches - 1) // n_batches + 1)])
        idx = torch.from_numpy(perm[: total * wl.batch].reshape(total, wl.batch).astype(np.int32)).to(m.device)
        lens_steps = lens[idx.long()].contiguous()                    # [total, batch] int32, built once, untimed
        step_ids = torch.arange(total, dtype=torch.int32, device=m.device)
        xbuf = torch.empty(wl.batch, wl.seq, wl.hidden, dtype=m.tdtype, device=m.device)
        lenbuf = torch.zeros(max(wl.batch, 64), dtype=torch.int32, device=m.device)
        row_bytes = wl.seq * wl.hidden * xbuf.element_size()
        len_row_bytes = wl.batch * 4
        assert len_row_bytes % 16 == 0
        st = side.cuda_stream

        def stage(t):
            B.mrem_gather_rows(calib, idx[t], wl.batch, row_bytes, xbuf, st)
            B.mrem_gather_rows(lens_steps, step_ids[t:t + 1], 1, len_row_bytes, lenbuf, st)

        stage(0)
        m.init_act_steps(xbuf, lenbuf, wl.batch, wl.seq)
        opt = B.make_optim(lr=wl.lr, step=0, decay_total_steps=max(wl.steps, W + K * max_repeats + 64))
        side.synchronize()
        B.mrem_graph_capture_step(m.ctx, xbuf, xbuf, 0.0, lenbuf, wl.batch, wl.seq, m.t_out, m.s_out, m.loss, opt)
        kernels_per_step = B.mrem_graph_num_kernels(m.ctx) + 2

        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for t in range(W):
            if t == W - 2:
                w0.record(side)
            stage(t)
            B.mrem_graph_launch(m.ctx)
        w1.record(side)
        side.synchronize()
        # timed blocks of exactly K steps each, every one bracketed by a barrier and a device synchronisation; enough of
        # them for a timed region of about 2 s (the last two warm-up steps give the estimate)
        repeats = args.repeats
        if repeats <= 0:
            est = D.max_over_ranks(w0.elapsed_time(w1) / 2, m.device)
            repeats = int(min(64, max(3, np.ceil(2000.0 / max(K * est, 1e-3)))))
        sampler = ClockSampler(local)
        block_ms = []
        for r in range(repeats):
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            if r == 0 and rank == 0:
                sampler.start()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for k in range(K):
                stage(W + (r * K + k) % (total - W))
                B.mrem_graph_launch(m.ctx)
            e1.record(side)
            side.synchronize()
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            block_ms.append(D.max_over_ranks(e0.elapsed_time(e1), m.device))
        clocks = sampler.stop() if rank == 0 else None
        ms = float(statistics.median(block_ms))
        loss_last = float(m.loss[0])
        status = m.poll_status()

        # ---- the same step captured on ONE stream (no kernel runs beside another): its replay time is the sum of the
        #      kernels' own run times plus their launch gaps, the cross-check of the per-kernel figures below
        serial_ms = None
        if world == 1:
            B.mrem_set_two_streams(m.ctx, 0)
            B.mrem_graph_capture_step(m.ctx, xbuf, xbuf, 0.0, lenbuf, wl.batch, wl.seq, m.t_out, m.s_out, m.loss, opt)
            for t in range(3):
                stage(W + t % (total - W))
                B.mrem_graph_launch(m.ctx)
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            side.synchronize()
            s0.record(side)
            for k in range(K):
                stage(W + k % (total - W))
                B.mrem_graph_launch(m.ctx)
            s1.record(side)
            side.synchronize()
            serial_ms = s0.elapsed_time(s1) / K
            B.mrem_set_two_streams(m.ctx, 1)
            B.mrem_graph_capture_step(m.ctx, xbuf, xbuf, 0.0, lenbuf, wl.batch, wl.seq, m.t_out, m.s_out, m.loss, opt)

        # ---- per-kernel timing (CUDA events around every launch of a few eager steps)
        B.mrem_trace_enable(m.ctx, 1)
        n_trace = 3
        for t in range(n_trace):
            stage(t)
            m.quantize_weights()
            m.forward_teacher(xbuf, lenbuf, wl.batch, wl.seq)
            m.forward_student(xbuf, lenbuf, wl.batch, wl.seq)
            m.recon_loss()
            m.backward()
            m.step(opt)
        trace = B.mrem_trace_read(m.ctx, 128)
        B.mrem_trace_enable(m.ctx, 0)

        # ---- end to end: host buffers in, loss out, every step
        e2e = None
        if not args.no_e2e:
            hb = [calib[idx[t].long()].cpu().pin_memory() for t in range(min(4, total))]
            hl = [lens_steps[t].cpu().pin_memory() for t in range(min(4, total))]
            ke = max(3, min(K, 50))
            for t in range(2):
                B.mrem_recon_step_host(m.ctx, hb[t % len(hb)], hb[t % len(hb)], hl[t % len(hl)], wl.batch, wl.seq, 0.0, opt)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            # submit / wait: the copy of batch t+1 from pinned host memory overlaps step t; every step still moves
            # its own inputs over PCIe and returns its own loss to the host
            B.mrem_recon_step_host_submit(m.ctx, hb[0], hb[0], hl[0], wl.batch, wl.seq, 0.0, opt)
            for t in range(1, ke):
                B.mrem_recon_step_host_submit(m.ctx, hb[t % len(hb)], hb[t % len(hb)], hl[t % len(hl)], wl.batch, wl.seq, 0.0, opt)
                loss_e2e = B.mrem_recon_step_host_wait(m.ctx)
            loss_e2e = B.mrem_recon_step_host_wait(m.ctx)
            torch.cuda.synchronize()
            dt_e2e = time.perf_counter() - t0
            dt_e2e = D.max_over_ranks(dt_e2e, m.device)
            e2e = {"value": D.whole_job_rate(tokens, ke, world, dt_e2e * 1e3), "unit": UNIT,
                   "h2d_bytes_per_step": row_bytes * wl.batch + len_row_bytes, "d2h_bytes_per_step": 4,
                   "steps": ke}
        extras = time_extras(m, wl, xbuf, lenbuf, side, torch, B, pk=peaks()) if args.extras and rank == 0 else None
        m.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    # products are traced per shape ("gemm_bf16 MxNxK.."); fold them into one row per kernel, keep the shapes
    # what an event pair measures around a kernel that does nothing: contained in every traced duration
    overhead_ms = 0.0
    for e in trace:
        if e["name"] == "(empty kernel)":
            overhead_ms = e["ms"] / max(e["launches"], 1)
    trace = [e for e in trace if e["name"] != "(empty kernel)"]
    net_ms = lambda e: max(e["ms"] - overhead_ms * e["launches"], 0.25 * e["ms"])
    shapes = [e for e in trace if e["name"].startswith("gemm_")]
    folded = {}
    for e in trace:
        key = {"gemm_bf16": "gemm_bf16_tcgen05", "gemm_i8": "gemm_i8_tcgen05"}.get(e["name"].split(" ")[0], e["name"])
        f = folded.setdefault(key, dict(name=key, ms=0.0, work=0.0, launches=0, is_flops=e["is_flops"]))
        f["ms"] += e["ms"]; f["work"] += e["work"]; f["launches"] += e["launches"]
    trace = list(folded.values())
    # Each launch is event-timed on its own; the denominator for the tensor-bound kernels is the burst figure when the
    # sampled SM clock sat at its maximum with no power cap (the conditions of a kernel timed alone), else the sustained one
    at_max = bool(clocks and clocks.get("sm_mhz") and clocks["sm_mhz"] >= 0.98 * clocks["sm_max_mhz"] and "sw_power_cap" not in clocks["reasons"])
    tensor_peak = "bf16_burst" if at_max else "bf16_sustained"
    kernels = []
    for e in sorted(trace, key=lambda e: -e["ms"]):
        per_launch_ms = e["ms"] / max(e["launches"], 1)
        e["net"] = net_ms(e)
        if e["is_flops"]:
            ach = e["work"] / (e["net"] * 1e-3) / 1e12
            peak = pk[tensor_peak] * (INT8_OVER_BF16 if "i8" in e["name"] else 1.0)
            unit, bound = "TFLOP/s", "tensor"
        else:
            ach = e["work"] / (e["net"] * 1e-3) / 1e9
            peak, unit, bound = pk["hbm_gbs"], "GB/s", "hbm"
        kernels.append({"name": e["name"], "launches_per_step": e["launches"] / n_trace, "ms_per_step": e["net"] / n_trace,
                        "us_per_launch": 1e3 * e["net"] / max(e["launches"], 1), "us_per_launch_with_event_overhead": 1e3 * per_launch_ms,
                        "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak})
    top = kernels[0]
    # DRAM bytes per launch of the dominant kernel from the committed ncu capture of this workload
    # (profiles/tc_gemm_dram_large6_w4a8.md); known only for that kernel on that workload
    traffic, traffic_file = ncu_dram_bytes_per_launch(wl.name, top["name"])
    roofline = {"kernel": top["name"], "bound": top["bound"], "achieved": top["achieved"], "peak": top["peak"],
                "unit": top["unit"], "frac": top["frac"], "traffic": traffic,
                "traffic_unit": f"bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum, ncu; {traffic_file})" if traffic else None,
                "peak_source": pk["source"] + ((" bf16 burst (SM clock at maximum, no power cap, during the run)" if at_max else
                                               " bf16 sustained (SM clock below maximum or power cap active during the run)")
                                              if top["bound"] == "tensor" else " copy bandwidth"),
                "int8_peak": "assumed: 2 x the measured bf16 figure (nominal dense ratio), not measured",
                "timed": f"CUDA events around each launch of {n_trace} eager steps, minus what the same event pair measures around a "
                         f"kernel that does nothing ({1e3 * overhead_ms:.2f} us, measured in this run); check: the kernels' net times "
                         f"add up to {sum(k['ms_per_step'] for k in kernels):.3f} ms per step, the step captured on one stream replays in "
                         f"{serial_ms if serial_ms is None else round(serial_ms, 3)} ms",
                "event_overhead_us": 1e3 * overhead_ms, "sum_net_ms_per_step": sum(k["ms_per_step"] for k in kernels),
                "serial_graph_ms_per_step": serial_ms}

    line = {"metric": METRIC, "value": D.whole_job_rate(tokens, K, world, ms), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": ms / K, "repeats": repeats, "ms_per_step_min": min(block_ms) / K,
            "timed_region_ms": sum(block_ms), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16+int8", "data": "synthetic",
            "config": workload_config(wl, calib_n, world),
            "clocks": clocks, "e2e": e2e, "gpu_launches": kernels_per_step * K * repeats, "roofline": roofline,
            "kernels": kernels,
            "gemm_shapes": [{"shape": e["name"], "launches_per_step": e["launches"] / n_trace,
                             "us_per_launch": 1e3 * net_ms(e) / max(e["launches"], 1),
                             "us_per_launch_with_event_overhead": 1e3 * e["ms"] / max(e["launches"], 1),
                             "tflops": e["work"] / (net_ms(e) * 1e-3) / 1e12} for e in sorted(shapes, key=lambda e: -e["ms"])],
            "loss_last": loss_last, "device_status": status}
    if extras:
        line["extras"] = extras
    if world == 1 and not args.no_cpu_baseline:
        val, threads, sample, sec = oracle_sample(wl)
        line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                                "seconds": sec}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
