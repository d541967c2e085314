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

# DRAM traffic per launch of the dominant kernel, from the ncu captures summarised under profiles/
# (dram__bytes_read.sum + dram__bytes_write.sum); None until a capture exists.
NCU_TRAFFIC_BYTES = {
    # profiles/block_decode_ring_kernel_config2.md: 274.2 MB on the B=128 capture, traffic is proportional to B
    "block_decode": 548.4e6,
    # profiles/block_decode_mq_kernel_dense_decode.md: 274.5 MB on the B=32 capture, traffic is proportional to B
    "dense_decode": 2196.0e6,
    # profiles/token_step_pipelined_kernel_config3.md: reads equal the algorithmic reads at j = 0 and j = 3 (25.2 + j x 16.8 MB);
    # the 25.2 MB written per launch mostly reach DRAM after the launch, so they are counted at their algorithmic size
    "token_decode": 75.5e6,
    # profiles/block_prefill_tc_kernel_config4.md: 110.5 MB inside the B=16 launch (reads exact, 9.7 of 33.5 MB of writes)
    "block_prefill": 221.0e6,
    "block_prefill_8k": None,
    "sweep": None,
}


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
    return c


# ------------------------------------------------------------------------------------------ GPU arm

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
    from paper_2406_02657_b200 import harness

    w = configs.sweep(args.block_len) if args.workload == "sweep" else configs.BY_NAME[args.workload]
    reduced = {}
    if args.batch:
        reduced["batch"] = args.batch
    if args.layers:
        reduced["n_layers"] = args.layers
    if args.prefix_len and args.workload == "token_decode" and args.prefix_len != w.prefix_len:
        w = configs.scaled(w, prefix_len=args.prefix_len)
    if reduced:  # a smaller copy of the workload, for profiler captures only
        w = configs.scaled(w, **reduced)
    fill = lambda tid, shape: gen.normal_bf16_device(replicas.replica_seed(w.seed, rank), tid, shape, device="cuda")
    pk = peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(step_fn, pre_fn, steps, warmup):
        """W untimed steps, then exactly K timed steps between barriers; returns ms per step (max over ranks)."""
        for _ in range(warmup):
            pre_fn()
            step_fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            pre_fn()
            step_fn()
        e1.record()
        barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1) / steps, world, device="cuda")

    sampler = ClockSampler(local_rank)
    kern_events = []
    if args.workload in ("block_decode", "block_decode_16k"):
        run = harness.BlockDecodeStep(w, fill=fill)
        tokens_per_step = w.batch * w.block_len
        # a bench step = one CUDA-graph replay of (put the lengths back, then 12 launches, each appending the
        # layer's new row and attending over the cache including it).
        # The per-launch time of the attention kernel comes from a twin graph of the same step with timing
        # events around every attention launch, replayed right after the timed region (events inside the
        # timed graph would lengthen the step they measure).
        run.capture()
        sampler.start()
        ms = timed(run.replay, lambda: None, args.steps, args.warmup)
        assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
        # the attention kernel's own launch time, two ways: (1) a graph of the 12 attention launches alone
        # (lengths as the step left them), which overlap their neighbours' ramp and drain exactly as in the
        # step: time / 12; (2) the twin graph with events, where every launch is fenced off by event nodes
        n_attn = max(10, min(args.steps, 50))
        ms_attn = timed(run.replay_attn, lambda: None, n_attn, 3) / w.n_layers
        for _ in range(3):
            run.replay_timed()
        torch.cuda.synchronize()
        kern_events = run.graph_events
        # end to end from pinned host buffers: rewind + bt_block_decode_step_host per layer (copies included),
        # captured once and replayed, so that the host's own speed does not enter the number
        run.capture_host()
        ms_e2e = timed(run.replay_host, lambda: None, args.steps, args.warmup)
        clocks = sampler.stop()  # sampled over the device-resident, the attention-only and the host-buffer runs
        h2d, d2h = run.host_bytes_per_step()
        alg_bytes = traffic.block_decode_layer_bytes(w.batch, w.heads, w.head_dim, w.ctx_blocks, with_append=False)
        dom = "block_decode_ring_kernel"
        launches = run.launches_per_step * args.steps
        step_bytes = w.n_layers * traffic.block_decode_layer_bytes(w.batch, w.heads, w.head_dim, w.ctx_blocks, True)
    elif args.workload == "dense_decode":
        run = harness.DenseDecodeStep(w, fill=fill)
        tokens_per_step = w.batch * w.block_len
        # a bench step = one CUDA-graph replay of (put the lengths back, then 12 launches, each appending the
        # block's L_B rows and running its L_B queries); per-launch time = step time / 12
        run.capture()
        sampler.start()
        ms = timed(run.replay, lambda: None, args.steps, args.warmup)
        clocks = sampler.stop()
        assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
        ms_e2e, h2d, d2h = None, 0, 0
        alg_bytes = traffic.dense_decode_layer_bytes(w.batch, w.heads, w.head_dim, w.ctx_blocks, w.block_len)
        dom = "block_decode_mq_kernel"
        launches = run.launches_per_step * args.steps
        step_bytes = w.n_layers * alg_bytes
    elif args.workload == "token_decode":
        run = harness.TokenDecodeRun(w, fill=fill)
        tokens_per_step = w.batch
        # a bench step = one CUDA-graph replay of `ring` token steps (a whole number of blocks), so that
        # every step does the same work and the 12 launches per token step are not host-bound
        n_tok = run.capture()
        sampler.start()
        ms_graph = timed(run.replay, lambda: None, args.steps, args.warmup)
        clocks = sampler.stop()
        assert run.status.item() == 0
        ms = ms_graph / n_tok
        ms_e2e, h2d, d2h = None, 0, 0
        P = w.prefix_len  # step 0 appends the P prefix rows, step j >= 1 one row over P + j - 1 cached rows
        alg_bytes = (traffic.token_decode_layer_bytes(w.batch, w.heads, w.head_dim, 0, P) +
                     sum(traffic.token_decode_layer_bytes(w.batch, w.heads, w.head_dim, P + j - 1) for j in range(1, w.block_len))) / w.block_len
        dom = "token_step_pipelined_kernel"
        launches = run.launches_per_step * n_tok * args.steps
        step_bytes = w.n_layers * alg_bytes
    elif args.workload == "sweep":
        # a bench step = one whole generation: prompt prefill + bulk append, then gen_tokens / L_B generated
        # blocks (CUDA-graph replays of `ring` blocks each); tokens = batch x generated tokens
        run = harness.GenerationRun(w, fill=fill)
        run.capture()
        tokens_per_step = w.batch * w.gen_tokens
        sampler.start()
        ms = timed(run.generate, lambda: None, args.steps, args.warmup)
        clocks = sampler.stop()
        assert run.status.item() == 0 and (run.block.len == w.max_blocks).all()
        ms_e2e, h2d, d2h = None, 0, 0
        parts = traffic.generation_bytes(w.batch, w.heads, w.head_dim, w.n_layers, w.block_len, w.prompt_tokens, w.gen_tokens)
        step_bytes = parts["total"]
        n_blocks = w.gen_tokens // w.block_len
        launches = (run.launches_prefill + run.launches_per_block * n_blocks) * args.steps
        dom = "block_decode_ring_kernel (whole generation: all kernels)"
        alg_bytes = step_bytes
        run.launches_per_step = 1  # the roofline line below is for the whole generation
    else:
        run = harness.PrefillRun(w, fill=fill)
        tokens_per_step = w.batch * w.prompt_tokens
        # a bench step = one CUDA-graph replay of the 12 launches (all of the same kernel, overlapping their
        # neighbours' ramp and drain through programmatic dependent launch); per-launch time = step time / 12
        run.capture()
        sampler.start()
        ms = timed(run.replay, lambda: None, args.steps, args.warmup)
        clocks = sampler.stop()
        kern_events = []
        ms_e2e, h2d, d2h = None, 0, 0
        alg_bytes = traffic.prefill_layer_bytes(w.batch, w.heads, w.prompt_blocks, w.head_dim)
        dom = "block_prefill_tc_kernel"
        launches = run.launches_per_step * args.steps
        step_bytes = w.n_layers * alg_bytes

    torch.cuda.synchronize()
    kern_ms_events = statistics.mean(a.elapsed_time(b) for a, b in kern_events) if kern_events else None
    if args.workload in ("block_decode", "block_decode_16k"):
        kern_ms = ms_attn
    elif kern_events:
        kern_ms = kern_ms_events
    else:
        kern_ms = ms / run.launches_per_step
    achieved = alg_bytes / (kern_ms * 1e-3) / 1e9
    roof = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / pk["hbm_gbs"], "peak_source": f"of {pk['_source']} (copy bandwidth)",
            "frac_of_8TBs_nominal": achieved / 8000.0, "kernel_ms": kern_ms, "kernel_ms_fenced_by_events": kern_ms_events, "algorithmic_bytes_per_launch": alg_bytes,
            "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
            "step_GBs": step_bytes / (ms * 1e-3) / 1e9}
    if args.workload.startswith("block_prefill"):
        fl = traffic.prefill_layer_flops(w.batch, w.heads, w.prompt_blocks, w.head_dim)
        roof["tensor_tflops"] = fl / (kern_ms * 1e-3) / 1e12
        roof["tensor_frac_of_measured_burst"] = roof["tensor_tflops"] / pk["bf16_tflops"]
        sustained = pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
        roof["tensor_frac_of_measured_sustained"] = roof["tensor_tflops"] / sustained
        if fl / alg_bytes > sustained * 1e12 / (pk["hbm_gbs"] * 1e9):
            # above the ridge (the 8K-prompt case): the tensor pipe is the binding roofline; the launches sit
            # inside a long step, so the sustained GEMM figure is the denominator
            roof.update(bound="tensor", hbm_GBs=achieved, achieved=roof["tensor_tflops"], peak=sustained, unit="TFLOP/s",
                        frac=roof["tensor_tflops"] / sustained, peak_source=f"of {pk['_source']} (sustained bf16 GEMM)")

    if rank != 0:
        return 0
    value = replicas.job_throughput(tokens_per_step, ms, world)
    if args.workload == "token_decode":
        ms, tokens_per_step = ms * n_tok, tokens_per_step * n_tok  # report the timed unit: one graph replay
    line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "accumulate": "f32", "data": "synthetic",
            "config": workload_config(w, args.workload), "clocks": clocks, "gpu_launches": launches,
            "roofline": roof}
    if ms_e2e is not None:
        line["e2e"] = {"value": replicas.job_throughput(tokens_per_step, ms_e2e, world), "unit": "tokens/s", "ms_per_step": ms_e2e,
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "api": "bt_block_decode_step_host, one call per layer spread over 3 streams (pinned host q,k,v in; out back to host; cache resident), the step captured in a CUDA graph and replayed"}
    if world == 1 and args.workload == "block_decode" and not args.no_cpu_baseline and not reduced:
        line["cpu_baseline"] = cpu_baseline_block_decode(w, run)
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
    ap.add_argument("--workload", default="block_decode", choices=["block_decode", "block_decode_16k", "dense_decode", "token_decode", "block_prefill", "block_prefill_8k", "sweep"])
    ap.add_argument("--block-len", type=int, default=4, help="L_B of the generation sweep (1, 2, 4 or 8)")
    ap.add_argument("--prefix-len", type=int, default=0, help="token_decode: prefix length P (default 1 = benchmark configs[2]; 2 = the paper's main setting)")
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
