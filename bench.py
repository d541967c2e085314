#!/usr/bin/env python
"""Benchmark of the Block Transformer KV-cache attention path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload block_decode|token_decode|block_prefill]
  python bench.py --impl reference ...      # times the CPU oracle instead (rank 0 only)

Default workload: the block-decoder decode step (batch 256, 16 heads, head_dim 64, L_B = 4,
2048-token context = 512 block-cache rows, 12 layers, each appending one row and attending).
One step advances every sequence by one block = L_B tokens.  Prints ONE JSON line.
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
sys.path.insert(0, ROOT)

from workloads import configs, gen, replicas, traffic  # noqa: E402

METRIC = "decode tokens/s (attention path)"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
            # nvidia-smi takes a few hundred ms to start: wait for its first sample so that short regions are covered
            t0 = time.time()
            while time.time() - t0 < 3.0 and os.path.getsize(self.path) == 0:
                time.sleep(0.02)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


dist_env = replicas.dist_env


# ------------------------------------------------------------------------------------------ CPU oracle legs

class OracleBlockDecodeSample:
    """The oracle on n_seq sequences of one layer of the block-decode step.  The inputs are drawn once;
    every step() puts the lengths back and times append + attention."""

    def __init__(self, w, n_seq, seed=None):
        import oracle
        seed = w.seed if seed is None else seed
        self.w, self.n_seq = w, n_seq
        B, H, hd, N = n_seq, w.heads, w.head_dim, w.max_blocks
        self.c = oracle.Cache(B, H, N, hd)
        self.c.k[...] = gen.normal_bf16_bits(seed, 0, self.c.k.shape)
        self.c.v[...] = gen.normal_bf16_bits(seed, 1, self.c.v.shape)
        self.q, self.k, self.v = (gen.normal_bf16_bits(seed, 2 + i, (B, H, 1, hd)) for i in range(3))
        self.q0 = np.ascontiguousarray(self.q[:, :, 0])
        oracle.lib()

    def step(self):
        """Returns the seconds the oracle took for one sample."""
        import oracle
        self.c.len[...] = self.w.ctx_blocks - 1
        t0 = time.perf_counter()
        oracle.kv_append(self.c, self.k, self.v)
        oracle.block_decode_attn(self.c, self.q0)
        return time.perf_counter() - t0


def cpu_baseline_block_decode(w, run):
    """The oracle on the whole step (all sequences, all layers), fed the bytes the GPU run used:
    each layer's cache is copied back to the host and handed to the oracle, which is timed alone."""
    import oracle
    oracle.lib()
    B, H, hd, N = w.batch, w.heads, w.head_dim, w.max_blocks
    secs = 0.0
    for l in range(w.n_layers):
        c = oracle.Cache(B, H, N, hd)
        c.k[...] = gen.torch_to_bits(run.cache.k[l])
        c.v[...] = gen.torch_to_bits(run.cache.v[l])
        c.len[...] = w.ctx_blocks - 1
        q, k, v = (gen.torch_to_bits(t[l]) for t in (run.q, run.k_new, run.v_new))
        t0 = time.perf_counter()
        oracle.kv_append(c, k, v)
        oracle.block_decode_attn(c, np.ascontiguousarray(q[:, :, 0]))
        secs += time.perf_counter() - t0
    tokens = w.batch * w.block_len
    return {"value": tokens / secs, "unit": "tokens/s", "cores": oracle.n_threads(), "kind": "oracle",
            "sample": f"one full step: {w.batch} sequences x {w.n_layers} layers (append + attention, fp64), "
                      f"{secs:.3f} s of oracle time, not scaled"}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the machine's host cores."""
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle
    if args.workload != "block_decode":
        print(json.dumps({"impl": "reference", "unavailable": "reference arm implemented for the block_decode workload only"}))
        return 0
    w = configs.BY_NAME[args.workload]
    n_seq = 64
    sample_run = OracleBlockDecodeSample(w, n_seq)
    for _ in range(max(1, min(args.warmup, 2))):
        sample_run.step()
    times = [sample_run.step() for _ in range(args.steps)]
    scale = (w.batch / n_seq) * w.n_layers
    step_s = statistics.mean(times) * scale
    tokens = w.batch * w.block_len
    val = tokens / step_s
    sample = f"per step: {n_seq} of {w.batch} sequences x 1 of {w.n_layers} layers, scaled x{scale:.0f}"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, args.workload),
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": oracle.n_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def workload_config(w, name):
    c = {"workload": name, "batch": w.batch, "heads": w.heads, "head_dim": w.head_dim, "block_len": w.block_len,
         "prefix_len": w.prefix_len, "n_layers": w.n_layers}
    if name == "block_decode":
        c.update(workload="block_decode: benchmark configs[1], per layer append 1 block row then attend over 512 rows",
                 ctx_blocks=w.ctx_blocks, context_tokens=w.ctx_blocks * w.block_len,
                 l2="no flush: 6.4 GB of KV per step, 537 MB per launch, L2 is 126 MB")
    elif name == "block_decode_16k":
        c.update(workload="block_decode_16k: the block-decoder decode step at a 16K-token context (4096 block rows), batch 64 "
                          "(with --batch 1..16: the small-batch case, row ranges split across the GPU)",
                 ctx_blocks=w.ctx_blocks, context_tokens=w.ctx_blocks * w.block_len,
                 l2="no flush: 1.07 GB of KV per launch at batch 64; at batch 1 a launch's 16.8 MB fit L2 but the 12 layers' 201 MB do not")
    elif name == "dense_decode":
        c.update(workload="dense_decode: the densified block decoder of the paper's future-work discussion - one cache row per "
                          "token (2048 rows), a step appends L_B = 4 rows and runs 4 queries per (sequence, head), 12 layers",
                 ctx_rows=w.ctx_blocks, context_tokens=w.ctx_blocks,
                 l2="no flush: 2.1 GB of KV per launch")
    elif name == "token_decode":
        c.update(workload="token_decode: benchmark configs[2], fused reset+append+local attention, 12 launches per token step",
                 l2="no flush: inputs rotate over a ring larger than L2")
    elif name == "sweep":
        c.update(workload=f"sweep: benchmark configs[4], decode-heavy generation at L_B = {w.block_len}: prompt {w.prompt_tokens} tokens, "
                          f"{w.gen_tokens} generated, block step every L_B tokens and token step every token",
                 prompt_tokens=w.prompt_tokens, gen_tokens=w.gen_tokens, max_blocks=w.max_blocks,
                 l2="no flush: the block cache alone is far larger than L2")
    elif name == "block_prefill_8k":
        c.update(workload="block_prefill_8k: the 8K-prompt case (2048 prompt blocks at L_B = 4, batch 8), same path as configs[3]",
                 prompt_blocks=w.prompt_blocks, l2="no flush: 3.2 GB of Q,K,V,out per step")
    elif name == "block_prefill":
        c.update(workload="block_prefill: benchmark configs[3], dense causal attention over 512 prompt blocks",
                 prompt_blocks=w.prompt_blocks, l2="no flush: 3.2 GB of Q,K,V,out per step")
    elif name == "qkv_project_token":
        c.update(workload="qkv_project_token: QKV projection of one token step at the shape of configs[2] (4096 rows, model dim 1024), "
                          "Q out, K and V rows written into the local cache by the epilogue, distinct weights per layer",
                 l2="no flush: 456 MB of inputs, weights and outputs per step, none of it reused")
    elif name == "qkv_project_block":
        c.update(workload="qkv_project_block: QKV projection of one block step at the shape of configs[1] (256 rows, model dim 1024), "
                          "K and V rows appended to the block cache by the epilogue, distinct weights per layer",
                 l2="no flush: the steps rotate over independent sets of inputs, weights and outputs, 288 MB per graph replay")
    elif name == "token_decode_projected":
        c.update(workload="token_decode_projected: configs[2] with the QKV projection in the path - per layer and token step, x [4096,1,1024] is "
                          "projected, K and V rows go into the local cache from the product's epilogue, the attention call attends over the "
                          "cache as it stands; 3 launches per layer and step (product, length update, attention)",
                 l2="no flush: inputs rotate over a ring larger than L2")
    elif name == "prefix_project":
        c.update(workload="prefix_project: context embedding -> P prefix embeddings for 4096 sequences, model dim 1024, 12 distinct weight sets",
                 l2="no flush: 250 MB per step")
    return c


# ------------------------------------------------------------------------------------------ GPU arm

# DRAM traffic per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture, summarised in the profiles folder), keyed by workload and, where it matters, prefix length.  A
# capture of a smaller batch is scaled by the batch ratio (traffic is proportional to the sequences
# processed).  None where no capture of the kernel as it stands exists.
NCU_TRAFFIC_BYTES = {
    ("block_decode", 1): 547.2e6,      # 273.6 MB captured at batch 128
    ("dense_decode", 1): 2196.0e6,     # 274.5 MB captured at batch 32
    # reads equal the algorithmic reads; the 25.2 MB written per launch mostly reach DRAM after the launch and
    # are counted at their algorithmic size
    ("token_decode", 1): 75.5e6,
    ("block_prefill", 1): 220.4e6,     # 110.2 MB captured at batch 16 (reads exact; 9-10 of 33.5 MB of writes reach DRAM inside the launch)
    ("block_prefill_8k", 1): 262.6e6,  # captured at full size: 216-218 MB read (Q, K, V are 201 MB), 45.5-46.5 of 67 MB written inside the launch
    # reads are x and W exactly once (14.7 MB); the 25.2 MB of q, K, V rows written stay in L2 until after the launch
    # and are counted at their algorithmic size
    ("qkv_project_token", 1): 39.9e6,
}


class Timer:
    """W untimed steps, then exactly K timed steps between barriers; ms per step, max over ranks."""

    def __init__(self, torch, dist, world):
        self.torch, self.dist, self.world = torch, dist, world

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def __call__(self, step_fn, steps, warmup):
        torch = self.torch
        for _ in range(warmup):
            step_fn()
        self.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step_fn()
        e1.record()
        self.barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1) / steps, self.world, device="cuda")


def hbm_roofline(pk, kernel, alg_bytes, launch_ms, step_bytes, step_ms, traffic_bytes, fenced_ms=None):
    achieved = alg_bytes / (launch_ms * 1e-3) / 1e9
    roof = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / pk["hbm_gbs"], "peak_source": f"of {pk['_source']} (copy bandwidth)",
            "frac_of_8TBs_nominal": achieved / 8000.0,
            # per-launch time = (time of a graph of the step's launches of this kernel) / launches: the launches
            # overlap their neighbours' ramp and drain through programmatic dependent launch, as inside the step
            "launch_ms_amortised_over_the_step": launch_ms,
            "algorithmic_bytes_per_launch": alg_bytes, "traffic": traffic_bytes,
            "step_GBs": step_bytes / (step_ms * 1e-3) / 1e9}
    if fenced_ms is not None:
        # the same launch fenced off by timing-event nodes on both sides (no overlap with its neighbours)
        roof["launch_ms_fenced_by_events"] = fenced_ms
        roof["frac_fenced"] = alg_bytes / (fenced_ms * 1e-3) / 1e9 / pk["hbm_gbs"]
    return roof


def add_tensor_roofline(roof, pk, flops, alg_bytes, launch_ms, in_long_step):
    """Tensor-pipe figures beside the HBM ones; above the ridge the tensor roofline becomes the reported bound."""
    tf = flops / (launch_ms * 1e-3) / 1e12
    burst, sustained = pk["bf16_tflops"], pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
    roof["tensor_tflops"] = tf
    roof["tensor_frac_of_measured_burst"] = tf / burst
    roof["tensor_frac_of_measured_sustained"] = tf / sustained
    roof["algorithmic_flops_per_launch"] = flops
    peak, which = (sustained, "sustained bf16 GEMM") if in_long_step else (burst, "burst bf16 GEMM")
    if flops / alg_bytes > peak * 1e12 / (pk["hbm_gbs"] * 1e9):
        roof.update(bound="tensor", hbm_GBs=roof["achieved"], achieved=tf, peak=peak, unit="TFLOP/s", frac=tf / peak,
                    peak_source=f"of {pk['_source']} ({which})")
    return roof


def oracle_sample(fn, tokens, what):
    """Times fn() (the oracle on a stated sample worth `tokens` tokens of the workload's metric)."""
    import oracle
    oracle.lib()
    t0 = time.perf_counter()
    fn()
    secs = time.perf_counter() - t0
    return {"value": tokens / secs, "unit": "tokens/s", "cores": oracle.n_threads(), "kind": "oracle",
            "sample": f"{what}; {secs:.2f} s of oracle time, scaled to the step"}


def measure(name, w, args, env, primary):
    """One workload: returns the fields of its JSON entry."""
    import torch
    from paper_2406_02657_b200 import harness
    timer, pk, fill, world, local_rank = env["timer"], env["pk"], env["fill"](w), env["world"], env["local_rank"]
    steps, warmup = args.steps, args.warmup
    sampler = ClockSampler(local_rank)
    out = {}
    e2e = None
    cpu = None
    P = w.prefix_len
    if name in ("block_decode", "block_decode_16k"):
        run = harness.BlockDecodeStep(w, fill=fill)
        tokens_per_step = w.batch * w.block_len
        # a step = one CUDA-graph replay of (put the lengths back, then one launch per layer, each appending the
        # layer's new row and attending over the cache including it)
        run.capture()
        sampler.start()
        ms = timer(run.replay, steps, warmup)
        assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
        # the attention kernel's own launch time, two ways: a graph of the attention launches alone (lengths as
        # the step left them), time / launches; and a twin graph of the step with timing events around every launch
        ms_attn = timer(run.replay_attn, max(10, min(steps, 50)), 3) / w.n_layers
        for _ in range(3):
            run.replay_timed()
        torch.cuda.synchronize()
        fenced = statistics.mean(a.elapsed_time(b) for a, b in run.graph_events)
        if primary:
            # end to end from pinned host buffers: rewind + bt_block_decode_step_host per layer (copies included),
            # captured once and replayed, so that the host's own speed does not enter the number
            run.capture_host()
            ms_e2e = timer(run.replay_host, steps, warmup)
            h2d, d2h = run.host_bytes_per_step()
            e2e = {"value": replicas.job_throughput(tokens_per_step, ms_e2e, world), "unit": "tokens/s", "ms_per_step": ms_e2e,
                   "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                   "api": "bt_block_decode_step_host, one call per layer spread over 3 streams (pinned host q,k,v in; out back to "
                          "host; cache resident), the step captured in a CUDA graph and replayed"}
        clocks = sampler.stop()
        alg = traffic.block_decode_layer_bytes(w.batch, w.heads, w.head_dim, w.ctx_blocks, with_append=False)
        step_bytes = w.n_layers * traffic.block_decode_layer_bytes(w.batch, w.heads, w.head_dim, w.ctx_blocks, True)
        roof = hbm_roofline(pk, "block_decode_ring_kernel", alg, ms_attn, step_bytes, ms,
                            NCU_TRAFFIC_BYTES.get((name, 1)) if w.batch == 256 else None, fenced)
        launches = run.launches_per_step * steps
        if primary and world == 1 and name == "block_decode" and not args.no_cpu_baseline and not env["reduced"]:
            cpu = cpu_baseline_block_decode(w, run)
    elif name == "dense_decode":
        run = harness.DenseDecodeStep(w, fill=fill)
        tokens_per_step = w.batch * w.block_len
        run.capture()
        sampler.start()
        ms = timer(run.replay, steps, warmup)
        clocks = sampler.stop()
        assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
        alg = traffic.dense_decode_layer_bytes(w.batch, w.heads, w.head_dim, w.ctx_blocks, w.block_len)
        roof = hbm_roofline(pk, "block_decode_mq_kernel", alg, ms / w.n_layers, w.n_layers * alg, ms,
                            NCU_TRAFFIC_BYTES.get((name, 1)) if w.batch == 256 else None)
        launches = run.launches_per_step * steps
    elif name == "token_decode":
        run = harness.TokenDecodeRun(w, fill=fill)
        # a step = one CUDA-graph replay of `ring` token steps (a whole number of blocks), so that every step
        # does the same work and the launches are not host-bound; reported per replay
        n_tok = run.capture()
        tokens_per_step = w.batch * n_tok
        sampler.start()
        ms = timer(run.replay, steps, warmup)
        clocks = sampler.stop()
        assert run.status.item() == 0
        # step 0 appends the P prefix rows, step j >= 1 one row over P + j - 1 cached rows
        alg = (traffic.token_decode_layer_bytes(w.batch, w.heads, w.head_dim, 0, P) +
               sum(traffic.token_decode_layer_bytes(w.batch, w.heads, w.head_dim, P + j - 1) for j in range(1, w.block_len))) / w.block_len
        n_launch = w.n_layers * n_tok
        roof = hbm_roofline(pk, "token_step_pipelined_kernel", alg, ms / n_launch, n_launch * alg, ms,
                            NCU_TRAFFIC_BYTES.get((name, P)) if w.batch == 4096 else None)
        launches = n_launch * steps
        if not primary and not args.no_cpu_baseline:
            import oracle
            n_seq, n_st = 256, 2 * w.block_len
            oc = oracle.Cache(n_seq, w.heads, w.local_cap, w.head_dim)
            sched = oracle.token_step_schedule(w.block_len, P, n_st)
            ins = [[gen.normal_bf16_bits(w.seed, 10 * t + i, (n_seq, w.heads, n_app, w.head_dim)) for i in range(3)] for t, (_, n_app, _) in enumerate(sched)]

            def go():
                for (reset, _, _), (q, k, v) in zip(sched, ins):
                    oracle.token_decode_attn(oc, q, k, v, reset_first=bool(reset))
            cpu = oracle_sample(go, n_seq * n_st / w.n_layers, f"{n_seq} of {w.batch} sequences x 1 of {w.n_layers} layers x {n_st} token steps")
    elif name == "token_decode_projected":
        run = harness.ProjectedTokenRun(w, fill=fill)
        n_tok = run.capture()
        tokens_per_step = w.batch * n_tok
        sampler.start()
        ms = timer(run.replay, steps, warmup)
        clocks = sampler.stop()
        assert run.status.item() == 0
        D = w.heads * w.head_dim
        # per layer and step: the product's bytes (x, W, bias in; q, K row, V row out) + the attention's (q in, the
        # j + 1 cached rows in, out out); the new K,V rows are written once, by the product
        row = w.head_dim * traffic.BF16
        attn = sum(w.batch * w.heads * (2 * row + (P + j) * 2 * row) for j in range(w.block_len)) / w.block_len
        alg = traffic.linear_bytes(w.batch, 3 * D, D) + attn
        fl = traffic.linear_flops(w.batch, 3 * D, D)
        n_layer_steps = w.n_layers * n_tok
        roof = hbm_roofline(pk, "project_tc_kernel + token_step_pipelined_kernel (one layer of one token step)", alg,
                            ms / n_layer_steps, n_layer_steps * alg, ms, None)
        add_tensor_roofline(roof, pk, fl, alg, ms / n_layer_steps, in_long_step=False)
        launches = run.launches_per_step * n_tok * steps
        if not args.no_cpu_baseline:
            import oracle
            n_seq, n_st = 32, w.block_len
            oc = oracle.Cache(n_seq, w.heads, w.local_cap, w.head_dim)
            xs = [gen.normal_bf16_bits(w.seed, 60 + t, (n_seq, 1, D)) for t in range(n_st)]
            Wq, bq = gen.normal_bf16_bits(w.seed, 70, (3 * D, D)), gen.normal_bf16_bits(w.seed, 71, (3 * D,))

            def go():
                for t in range(n_st):
                    q = oracle.qkv_project_append(oc, xs[t], Wq, bq, reset_first=(t == 0))
                    oracle.token_decode_attn(oc, oracle.round_to_bf16(q), None, None)
            cpu = oracle_sample(go, n_seq * n_st / w.n_layers, f"{n_seq} of {w.batch} sequences x 1 of {w.n_layers} layers x {n_st} token steps "
                                                              f"(projection + append + attention, fp64)")
    elif name == "sweep":
        # a step = one whole generation: prompt prefill + bulk append, then gen_tokens / L_B generated blocks
        # (CUDA-graph replays of `ring` blocks each); tokens = batch x generated tokens
        run = harness.GenerationRun(w, fill=fill)
        run.capture()
        tokens_per_step = w.batch * w.gen_tokens
        sampler.start()
        ms = timer(run.generate, steps, warmup)
        clocks = sampler.stop()
        assert run.status.item() == 0 and (run.block.len == w.max_blocks).all()
        parts = traffic.generation_bytes(w.batch, w.heads, w.head_dim, w.n_layers, w.block_len, w.prompt_tokens, w.gen_tokens)
        n_blocks = w.gen_tokens // w.block_len
        launches = (run.launches_prefill + run.launches_per_block * n_blocks) * steps
        roof = hbm_roofline(pk, "whole generation: all kernels", parts["total"], ms, parts["total"], ms, None)
        roof["bytes_by_part"] = parts
        if not args.no_cpu_baseline:
            import oracle
            n_seq, n_blk, rows = 4, 8, w.prompt_blocks + n_blocks // 2   # taken at the middle of the generation
            bc = oracle.Cache(n_seq, w.heads, w.max_blocks, w.head_dim)
            bc.k[...], bc.v[...] = (gen.normal_bf16_bits(w.seed, i, bc.k.shape) for i in (0, 1))
            bc.len[...] = rows
            lcache = oracle.Cache(n_seq, w.heads, w.local_cap, w.head_dim)
            ins = [gen.normal_bf16_bits(w.seed, 2 + i, (n_seq, w.heads, 1, w.head_dim)) for i in range(3)]

            def go():
                for _ in range(n_blk):
                    for j in range(w.block_len):
                        oracle.token_decode_attn(lcache, *ins, reset_first=(j == 0))
                    oracle.kv_append(bc, ins[1], ins[2])
                    oracle.block_decode_attn(bc, np.ascontiguousarray(ins[0][:, :, 0]))
            cpu = oracle_sample(go, n_seq * n_blk * w.block_len / w.n_layers,
                                f"{n_seq} of {w.batch} sequences x 1 of {w.n_layers} layers of each decoder x {n_blk} generated blocks at the "
                                f"middle of the generation ({rows} cached blocks); the prompt's prefill is left out")
    elif name in ("qkv_project_token", "qkv_project_block", "prefix_project"):
        kind = {"qkv_project_token": "qkv_token", "qkv_project_block": "qkv_block", "prefix_project": "prefix"}[name]
        # enough independent weight sets that one graph replay moves more than the 126 MB L2 holds
        per_set = w.n_layers * traffic.linear_bytes(w.batch, (3 if kind != "prefix" else P) * w.heads * w.head_dim, w.heads * w.head_dim)
        sets = max(1, -(-(200 << 20) // per_set))
        run = harness.ProjectRun(w, kind, fill=fill, sets=sets)
        tokens_per_step = w.batch * (w.block_len if kind == "qkv_block" else 1)
        run.capture()
        sampler.start()
        ms = timer(run.replay, steps, warmup) / sets   # a replay is `sets` steps
        clocks = sampler.stop()
        assert run.status.item() == 0
        alg = traffic.linear_bytes(run.M, run.N, run.K)
        fl = traffic.linear_flops(run.M, run.N, run.K)
        roof = hbm_roofline(pk, "project_tc_kernel", alg, ms / w.n_layers, w.n_layers * alg, ms,
                            NCU_TRAFFIC_BYTES.get((name, 1)) if w.batch == 4096 else None)
        add_tensor_roofline(roof, pk, fl, alg, ms / w.n_layers, in_long_step=False)
        launches = run.launches_per_step * steps
        if not args.no_cpu_baseline:
            import oracle
            rows = 64
            x, W, b = (gen.normal_bf16_bits(w.seed, i, sh) for i, sh in enumerate(((rows, run.K), (run.N, run.K), (run.N,))))
            cpu = oracle_sample(lambda: oracle.linear(x, W, b), tokens_per_step * rows / run.M / w.n_layers,
                                f"{rows} of {run.M} rows x 1 of {w.n_layers} layers (y = W x + b in fp64)")
    else:  # block_prefill, block_prefill_8k
        run = harness.PrefillRun(w, fill=fill)
        tokens_per_step = w.batch * w.prompt_tokens
        # a step = one CUDA-graph replay of the launches of all layers (the same kernel, overlapping their
        # neighbours' ramp and drain through programmatic dependent launch); per-launch time = step time / layers
        run.capture()
        sampler.start()
        ms = timer(run.replay, steps, warmup)
        clocks = sampler.stop()
        alg = traffic.prefill_layer_bytes(w.batch, w.heads, w.prompt_blocks, w.head_dim)
        fl = traffic.prefill_layer_flops(w.batch, w.heads, w.prompt_blocks, w.head_dim)
        roof = hbm_roofline(pk, "block_prefill_tc_kernel", alg, ms / w.n_layers, w.n_layers * alg, ms,
                            NCU_TRAFFIC_BYTES.get((name, 1)) if w.batch == configs.BY_NAME[name].batch else None)
        add_tensor_roofline(roof, pk, fl, alg, ms / w.n_layers, in_long_step=True)
        launches = run.launches_per_step * steps
        if not primary and not args.no_cpu_baseline:
            import oracle
            n_h = 2
            q, k, v = (gen.normal_bf16_bits(w.seed, i, (1, n_h, w.prompt_blocks, w.head_dim)) for i in range(3))
            cpu = oracle_sample(lambda: oracle.block_prefill_attn(q, k, v), w.prompt_tokens * n_h / w.heads / w.n_layers,
                                f"1 of {w.batch} sequences x {n_h} of {w.heads} heads x 1 of {w.n_layers} layers")
    del run
    torch.cuda.empty_cache()
    out.update(value=replicas.job_throughput(tokens_per_step, ms, world), unit="tokens/s", ms_per_step=ms, steps=steps, warmup=warmup,
               config=workload_config(w, name), clocks=clocks, gpu_launches=launches, roofline=roof)
    if e2e is not None:
        out["e2e"] = e2e
    if cpu is not None:
        out["cpu_baseline"] = cpu
    return out


# what the default run measures after its primary line: (workload, prefix length, block length, steps, warm-up)
SECONDARY = [
    # step counts sized for about half a second of timed work each, so that the clock sampler sees the region
    ("token_decode", 1, 0, 400, 3), ("token_decode", 2, 0, 300, 3), ("token_decode", 8, 0, 150, 3), ("block_prefill", 0, 0, 600, 3), ("block_prefill_8k", 0, 0, 250, 3),
    ("qkv_project_token", 0, 0, 1200, 3), ("qkv_project_block", 0, 0, 2000, 3), ("prefix_project", 0, 0, 2000, 3),
    ("token_decode_projected", 0, 0, 120, 3),
    ("sweep", 0, 4, 2, 1), ("sweep", 0, 8, 2, 1),
]


def run_gpu(args):
    import torch
    import torch.distributed as dist

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    import paper_2406_02657_b200 as bt  # noqa: F401  (loads libbt.so; raises if it cannot)

    w = configs.sweep(args.block_len) if args.workload == "sweep" else configs.BY_NAME[args.workload]
    reduced = {}
    if args.batch:
        reduced["batch"] = args.batch
    if args.layers:
        reduced["n_layers"] = args.layers
    if args.prefix_len and args.prefix_len != w.prefix_len:
        w = configs.scaled(w, prefix_len=args.prefix_len)
    if reduced:  # a smaller copy of the workload, for profiler captures only
        w = configs.scaled(w, **reduced)
    env = {"timer": Timer(torch, dist, world), "pk": peaks(), "world": world, "local_rank": local_rank, "reduced": reduced,
           "fill": lambda wl: (lambda tid, shape: gen.normal_bf16_device(replicas.replica_seed(wl.seed, rank), tid, shape, device="cuda"))}
    m = measure(args.workload, w, args, env, primary=True)
    secondary = {}
    if world == 1 and args.workload == "block_decode" and not reduced and not args.no_secondary:
        # the other configurations, shorter runs of the same measurement, under one key of the same line
        for name, P, L_B, k, wu in SECONDARY:
            ws = configs.sweep(L_B) if name == "sweep" else configs.BY_NAME[name]
            if P and P != ws.prefix_len:
                ws = configs.scaled(ws, prefix_len=P)
            a2 = argparse.Namespace(**vars(args))
            a2.steps, a2.warmup = k, wu
            key = name + (f"_P{P}" if P else "") + (f"_LB{L_B}" if L_B else "")
            secondary[key] = measure(name, ws, a2, env, primary=False)
    if rank == 0:
        line = {"metric": METRIC, "value": m["value"], "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "accumulate": "f32", "data": "synthetic",
                "config": m["config"], "clocks": m["clocks"], "gpu_launches": m["gpu_launches"], "roofline": m["roofline"]}
        for key in ("e2e", "cpu_baseline"):
            if key in m:
                line[key] = m[key]
        if secondary:
            line["secondary"] = secondary
        if reduced:
            line["reduced_case_not_a_bench_number"] = reduced
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps (default 200; 3 for the sweep, whose step is a whole generation)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="block_decode",
                    choices=["block_decode", "block_decode_16k", "dense_decode", "token_decode", "block_prefill", "block_prefill_8k", "sweep",
                             "qkv_project_token", "qkv_project_block", "prefix_project", "token_decode_projected"])
    ap.add_argument("--no-secondary", action="store_true", help="default workload only: skip the shorter runs of the other configurations")
    ap.add_argument("--block-len", type=int, default=4, help="L_B of the generation sweep (1, 2, 4 or 8)")
    ap.add_argument("--prefix-len", type=int, default=0, help="prefix length P (token_decode: default 1 = benchmark configs[2], 2 = the paper's main setting; prefix_project: default 2)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the batch (profiling a small case; not a bench number)")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling a small case)")
    args = ap.parse_args()
    if args.steps <= 0:
        args.steps = 3 if args.workload == "sweep" else 200
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
