"""Synthetic drivers for the paper's serving workloads (section 3.2: prompts padded to one length,
prefill-heavy 2048/128 and decode-heavy 128/2048): they own the device buffers and issue the
library calls of one step.  No arithmetic of the method happens here.
"""
from __future__ import annotations

import torch

from . import binding as bt


class BlockDecodeStep:
    """One block-decoder decode step over all layers (section 2.3): per layer, append the new
    block's K,V row, then attend causally over the whole block cache - one fused launch per
    layer (bt_block_decode_step), or with ``fused=False`` the two separate calls.

    The caches are pre-filled to ``ctx_blocks - 1`` rows so that after the append every sequence
    attends over ``ctx_blocks`` rows.  ``rewind()`` puts the lengths back so a step can be repeated.
    """

    def __init__(self, w, device="cuda", fill=None, fused=True):
        self.w, self.device, self.fused = w, device, fused
        self.cfg = bt.make_config(w.batch, w.heads, w.head_dim, w.block_len, w.prefix_len, w.max_blocks, w.n_layers)
        shape = (w.n_layers, w.batch, w.heads, w.max_blocks, w.head_dim)
        if fill is None:
            k = torch.zeros(shape, dtype=torch.bfloat16, device=device)
            v = torch.zeros(shape, dtype=torch.bfloat16, device=device)
        else:
            k, v = fill(0, shape), fill(1, shape)
        self.cache = bt.BlockCache(self.cfg, device, k=k, v=v)
        self.len0 = torch.full((w.n_layers, w.batch), w.ctx_blocks - 1, dtype=torch.int32, device=device)
        self.cache.len.copy_(self.len0)
        io = (w.n_layers, w.batch, w.heads, 1, w.head_dim)
        mk = (lambda tid: fill(tid, io)) if fill is not None else (lambda tid: torch.zeros(io, dtype=torch.bfloat16, device=device))
        self.q, self.k_new, self.v_new = mk(2), mk(3), mk(4)
        self.out = torch.empty(io, dtype=torch.bfloat16, device=device)
        self.ws = bt.alloc_workspace(self.cfg, device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        # per layer one fused launch, or append + attention (split row ranges are merged inside the launch)
        self.launches_per_step = w.n_layers * (1 if fused else 2)
        self._host = None

    def rewind(self):
        self.cache.len.copy_(self.len0, non_blocking=True)

    def step(self, attn_events=None):
        """Enqueue one step.  attn_events: optional list receiving (start, stop) CUDA events around
        each attention launch."""
        for l in range(self.w.n_layers):
            if not self.fused:
                bt.bt_block_kv_append(self.cfg, self.cache, l, self.k_new[l], self.v_new[l], n_new=1, dev_status=self.status)
            if attn_events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            self._layer(l)
            if attn_events is not None:
                e1.record()
                attn_events.append((e0, e1))

    def _layer(self, l):
        """The attention launch of layer l: with the append fused in, or after a separate append."""
        if self.fused:
            bt.bt_block_decode_step(self.cfg, self.cache, l, self.q[l], self.k_new[l], self.v_new[l], self.out[l], self.ws,
                                    dev_status=self.status)
        else:
            bt.bt_block_decode_attn(self.cfg, self.cache, l, self.q[l], self.out[l], self.ws, dev_status=self.status)

    def _capture(self, events):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.rewind()
            for l in range(self.w.n_layers):
                if not self.fused:
                    bt.bt_block_kv_append(self.cfg, self.cache, l, self.k_new[l], self.v_new[l], n_new=1, dev_status=self.status)
                if events is not None:
                    e0 = torch.cuda.Event(enable_timing=True, external=True)
                    e1 = torch.cuda.Event(enable_timing=True, external=True)
                    e0.record()
                self._layer(l)
                if events is not None:
                    e1.record()
                    events.append((e0, e1))
        return g

    def capture(self):
        """Capture rewind + one whole step into CUDA graphs: a plain one (replay), one with timing events
        (external, so that they may sit inside a graph) around every attention launch (replay_timed;
        after it the events hold that replay's per-launch times), and the attention launches alone
        (replay_attn)."""
        self.step()  # anything lazy (module load, per-device set-up) happens outside the capture
        self.rewind()
        torch.cuda.synchronize()
        self.graph = self._capture(None)
        self.graph_events = []
        self.graph_timed = self._capture(self.graph_events)
        # the attention launches alone (lengths as a step leaves them: ctx_blocks rows), for their own time
        self.graph_attn = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_attn):
            for l in range(self.w.n_layers):
                bt.bt_block_decode_attn(self.cfg, self.cache, l, self.q[l], self.out[l], self.ws, dev_status=self.status)

    def replay_attn(self):
        self.graph_attn.replay()

    def replay_timed(self):
        self.graph_timed.replay()

    def replay(self):
        self.graph.replay()

    # ---- the same step driven from pinned host buffers through bt_block_decode_step_host
    def _host_buffers(self):
        if self._host is None:
            pin = lambda t: t.cpu().pin_memory()
            self._host = dict(q=pin(self.q), k=pin(self.k_new), v=pin(self.v_new), out=torch.empty_like(self.out, device="cpu").pin_memory(),
                              qd=torch.empty_like(self.q), kd=torch.empty_like(self.k_new), vd=torch.empty_like(self.v_new))
        return self._host

    def host_bytes_per_step(self):
        one = self.w.batch * self.w.heads * self.w.head_dim * 2
        return 3 * one * self.w.n_layers, one * self.w.n_layers

    def step_host(self, n_streams=3):
        """The step through bt_block_decode_step_host, one call per layer.  The layers' inputs all come from
        the host, so the calls are independent: they are spread round-robin over a few streams (forked from
        and joined back into the current one), which lets one layer's host-device copies run under another
        layer's kernels.  Each stream has its own workspace (the calls of one stream are ordered)."""
        h = self._host_buffers()
        main = torch.cuda.current_stream()
        if getattr(self, "_side", None) is None or len(self._side) != n_streams:
            self._side = [torch.cuda.Stream() for _ in range(n_streams)]
            self._side_ws = [bt.alloc_workspace(self.cfg, self.device) for _ in range(n_streams)]
            self._fork = torch.cuda.Event()
            self._join = [torch.cuda.Event() for _ in range(n_streams)]
        self._fork.record(main)
        for s in self._side:
            s.wait_event(self._fork)
        for l in range(self.w.n_layers):
            i = l % n_streams
            bt.bt_block_decode_step_host(self.cfg, self.cache, l, h["q"][l], h["k"][l], h["v"][l], h["out"][l],
                                         h["qd"][l], h["kd"][l], h["vd"][l], self.out[l], self._side_ws[i], dev_status=self.status,
                                         stream=self._side[i])
        for s, e in zip(self._side, self._join):
            e.record(s)
            main.wait_event(e)


    def capture_host(self, n_streams=3):
        """Capture rewind + step_host (the copies from and to pinned host memory included) into a CUDA graph,
        so that a step costs the host one launch instead of some sixty API calls; replay_host() runs it."""
        self._host_buffers()
        self.rewind()
        self.step_host(n_streams)   # creates the side streams, their workspaces and events outside the capture
        self.rewind()
        torch.cuda.synchronize()
        self.graph_host = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_host):
            self.rewind()
            self.step_host(n_streams)

    def replay_host(self):
        self.graph_host.replay()


class DenseDecodeStep:
    """One step of the densified block decoder over all layers (the paper's discussion of future work):
    per layer one launch appends the block's L_B sub-block rows and runs its L_B queries over the
    cache.  The caches are pre-filled so that after the append every sequence holds ``ctx_blocks`` rows."""

    def __init__(self, w, device="cuda", fill=None):
        self.w, self.device = w, device
        m = w.block_len
        self.cfg = bt.make_config(w.batch, w.heads, w.head_dim, w.block_len, w.prefix_len, w.max_blocks, w.n_layers)
        shape = (w.n_layers, w.batch, w.heads, w.max_blocks, w.head_dim)
        mk = fill if fill is not None else (lambda tid, sh: torch.zeros(sh, dtype=torch.bfloat16, device=device))
        self.cache = bt.BlockCache(self.cfg, device, k=mk(0, shape), v=mk(1, shape))
        self.len0 = torch.full((w.n_layers, w.batch), w.ctx_blocks - m, dtype=torch.int32, device=device)
        self.cache.len.copy_(self.len0)
        io = (w.n_layers, w.batch, w.heads, m, w.head_dim)
        self.q, self.k_new, self.v_new = mk(2, io), mk(3, io), mk(4, io)
        self.out = torch.empty(io, dtype=torch.bfloat16, device=device)
        self.ws = bt.alloc_workspace(self.cfg, device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.launches_per_step = w.n_layers
        self.graph = None

    def rewind(self):
        self.cache.len.copy_(self.len0, non_blocking=True)

    def step(self):
        for l in range(self.w.n_layers):
            bt.bt_block_decode_step_multi(self.cfg, self.cache, l, self.q[l], self.k_new[l], self.v_new[l], self.out[l], self.ws,
                                          dev_status=self.status)

    def capture(self):
        self.step()  # anything lazy happens outside the capture
        self.rewind()
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.rewind()
            self.step()

    def replay(self):
        self.graph.replay()


class TokenDecodeRun:
    """Token-decoder steps over all layers (section 2.4): step 0 of a block resets the local cache and
    appends the P prefix rows (P queries, causal among themselves), step j >= 1 appends the row of the
    token produced by step j-1; every step attends over the local cache (prefix + tokens of the same
    block)."""

    def __init__(self, w, device="cuda", fill=None, ring=8):
        self.w, self.device = w, device
        self.cfg = bt.make_config(w.batch, w.heads, w.head_dim, w.block_len, w.prefix_len, max(1, w.max_blocks), w.n_layers)
        self.cache = bt.LocalCache(self.cfg, device)
        P = w.prefix_len
        io = (ring, w.n_layers, w.batch, w.heads, P, w.head_dim)  # step 0 of a block uses all P rows, later steps row 0
        mk = (lambda tid: fill(tid, io)) if fill is not None else (lambda tid: torch.zeros(io, dtype=torch.bfloat16, device=device))
        self.q, self.k_new, self.v_new = mk(5), mk(6), mk(7)
        self.out = torch.empty(io[1:], dtype=torch.bfloat16, device=device)
        # contiguous one-row views for the steps after the first (the library takes [B][H][n][hd] contiguous)
        if P > 1:
            self.q1, self.k1, self.v1 = (t[:, :, :, :, :1].contiguous() for t in (self.q, self.k_new, self.v_new))
            self.out1 = torch.empty((w.n_layers, w.batch, w.heads, 1, w.head_dim), dtype=torch.bfloat16, device=device)
        else:
            self.q1, self.k1, self.v1, self.out1 = self.q, self.k_new, self.v_new, self.out
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.ring = ring
        self.t = 0
        self.launches_per_step = w.n_layers

    def token_step(self, events=None):
        """Token step t.  events: optional list receiving an (external) timing event pair around every launch."""
        w = self.w
        j = self.t % w.block_len
        r = self.t % self.ring
        first = j == 0
        q, k, v, out = (self.q, self.k_new, self.v_new, self.out) if first else (self.q1, self.k1, self.v1, self.out1)
        for l in range(w.n_layers):
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True, external=True)
                e1 = torch.cuda.Event(enable_timing=True, external=True)
                e0.record()
            bt.bt_token_decode_attn(self.cfg, self.cache, l, q[r, l], k[r, l], v[r, l], out[l],
                                    n_q=(w.prefix_len if first else 1), reset_first=first, dev_status=self.status)
            if events is not None:
                e1.record()
                events.append((e0, e1))
        self.t += 1

    def capture(self, n_steps=None):
        """Capture n_steps consecutive token steps (default: one pass over the input ring, a whole
        number of blocks) into a CUDA graph; replay() then advances the run by that many steps."""
        n_steps = self.ring if n_steps is None else n_steps
        assert n_steps % self.w.block_len == 0 and self.t % self.w.block_len == 0
        self.token_step()  # make sure nothing lazy (module load) happens inside the capture
        self.t -= 1
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            for _ in range(n_steps):
                self.token_step()
        self.graph_steps = n_steps
        return n_steps

    def replay(self):
        self.graph.replay()


class PrefillRun:
    """Block-decoder prefill over all layers (sections 2.1, 2.3): dense causal attention over the
    T prompt blocks, distinct Q, K, V, out per layer."""

    def __init__(self, w, device="cuda", fill=None):
        self.w = w
        self.cfg = bt.make_config(w.batch, w.heads, w.head_dim, w.block_len, w.prefix_len, w.max_blocks, w.n_layers)
        shape = (w.n_layers, w.batch, w.heads, w.prompt_blocks, w.head_dim)
        mk = (lambda tid: fill(tid, shape)) if fill is not None else (lambda tid: torch.zeros(shape, dtype=torch.bfloat16, device=device))
        self.q, self.k, self.v = mk(8), mk(9), mk(10)
        self.out = torch.empty(shape, dtype=torch.bfloat16, device=device)
        self.launches_per_step = w.n_layers

    def capture(self):
        """One step as two CUDA graphs: a plain one (replay) and a twin with (external) timing events
        around every launch (replay_timed; afterwards graph_events hold that replay's times)."""
        self.step()
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.step()
        self.graph_events = []
        self.graph_timed = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_timed):
            self.step(self.graph_events, external=True)

    def replay(self):
        self.graph.replay()

    def replay_timed(self):
        self.graph_timed.replay()

    def step(self, events=None, external=False):
        for l in range(self.w.n_layers):
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True, external=external), torch.cuda.Event(enable_timing=True, external=external)
                e0.record()
            bt.bt_block_prefill_attn(self.cfg, self.q[l], self.k[l], self.v[l], self.out[l], n_blocks=self.w.prompt_blocks)
            if events is not None:
                e1.record()
                events.append((e0, e1))


class GenerationRun:
    """Decode-heavy generation (section 3.2: 128-token prompt, 2048 generated tokens) through both
    decoders' attention: prefill of the prompt's T blocks and bulk append of their K,V rows, then per
    generated block L_B token-decoder steps (reset at the first) and one block-decoder step (append
    one row, attend over all rows), n_layers each.  Step inputs rotate over a small ring of
    pre-drawn tensors; one pass over the ring is captured as a CUDA graph and replayed."""

    def __init__(self, w, device="cuda", fill=None, ring=4):
        self.w, self.device, self.ring = w, device, ring
        L, B, H, hd = w.n_layers, w.batch, w.heads, w.head_dim
        self.cfg = bt.make_config(B, H, hd, w.block_len, w.prefix_len, w.max_blocks, L)
        mk = (lambda tid, shape: fill(tid, shape)) if fill is not None else \
            (lambda tid, shape: torch.zeros(shape, dtype=torch.bfloat16, device=device))
        T = w.prompt_blocks
        self.pq, self.pk, self.pv = (mk(20 + i, (L, B, H, T, hd)) for i in range(3))
        self.pout = torch.empty((L, B, H, T, hd), dtype=torch.bfloat16, device=device)
        self.bq, self.bk, self.bv = (mk(23 + i, (ring, L, B, H, 1, hd)) for i in range(3))
        self.bout = torch.empty((L, B, H, 1, hd), dtype=torch.bfloat16, device=device)
        self.tq, self.tk, self.tv = (mk(26 + i, (ring, w.block_len, L, B, H, 1, hd)) for i in range(3))
        self.tout = torch.empty((L, B, H, 1, hd), dtype=torch.bfloat16, device=device)
        self.block = bt.BlockCache(self.cfg, device, k=torch.empty((L, B, H, w.max_blocks, hd), dtype=torch.bfloat16, device=device),
                                   v=torch.empty((L, B, H, w.max_blocks, hd), dtype=torch.bfloat16, device=device))
        self.local = bt.LocalCache(self.cfg, device)
        self.ws = bt.alloc_workspace(self.cfg, device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.n_gen_blocks = w.gen_tokens // w.block_len
        self.graph = None
        self.launches_prefill = 2 * L
        self.launches_per_block = L * (w.block_len + 1)   # L_B token steps + one fused block step, per layer

    def start(self):
        """Empty caches, then the prompt: prefill attention and bulk append per layer."""
        self.block.len.zero_()
        self.local.len.zero_()
        w = self.w
        for l in range(w.n_layers):
            bt.bt_block_prefill_attn(self.cfg, self.pq[l], self.pk[l], self.pv[l], self.pout[l], n_blocks=w.prompt_blocks,
                                     dev_status=self.status)
            bt.bt_block_kv_append(self.cfg, self.block, l, self.pk[l], self.pv[l], n_new=w.prompt_blocks, dev_status=self.status)

    def gen_block(self, r):
        """One generated block with ring slot r: L_B token steps, then the block step."""
        w = self.w
        for j in range(w.block_len):
            for l in range(w.n_layers):
                bt.bt_token_decode_attn(self.cfg, self.local, l, self.tq[r, j, l], self.tk[r, j, l], self.tv[r, j, l], self.tout[l],
                                        n_q=1, reset_first=(j == 0), dev_status=self.status)
        for l in range(w.n_layers):
            bt.bt_block_decode_step(self.cfg, self.block, l, self.bq[r, l], self.bk[r, l], self.bv[r, l], self.bout[l], self.ws,
                                    dev_status=self.status)

    def capture(self):
        """One pass over the input ring (ring generated blocks) as a CUDA graph."""
        assert self.n_gen_blocks % self.ring == 0
        self.start()
        self.gen_block(0)  # anything lazy happens outside the capture
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            for r in range(self.ring):
                self.gen_block(r)

    def generate(self):
        """The whole generation: prompt, then n_gen_blocks generated blocks (graph replays)."""
        self.start()
        if self.graph is None:
            for g in range(self.n_gen_blocks):
                self.gen_block(g % self.ring)
        else:
            for _ in range(self.n_gen_blocks // self.ring):
                self.graph.replay()


class ProjectRun:
    """The linear maps either side of the attention path over all layers, with distinct weights per layer:
    kind "qkv_token" - one token step of the token decoder (section 2.4): x [B,1,D] -> q, K and V rows into
    the local cache (reset at every launch so that a step can be repeated); kind "qkv_block" - one block
    step of the block decoder (section 2.3): x [B,1,D] -> q, K and V rows appended to the block cache (the
    lengths are put back before every step); kind "prefix" - context embedding [B,D] -> P prefix embeddings.
    ``sets`` independent copies of the per-layer tensors are used round-robin, `sets` steps per graph replay,
    so that a replay's working set can be made larger than the L2 cache."""

    def __init__(self, w, kind, device="cuda", fill=None, sets=1):
        self.w, self.kind, self.sets = w, kind, sets
        B, H, hd, P = w.batch, w.heads, w.head_dim, w.prefix_len
        L = w.n_layers * sets   # tensors are [sets * layers, ...]; set s uses rows s*layers .. (s+1)*layers-1
        D = H * hd
        self.cfg = bt.make_config(B, H, hd, w.block_len, P, max(1, w.max_blocks), w.n_layers)
        mk = fill if fill is not None else (lambda tid, sh: torch.zeros(sh, dtype=torch.bfloat16, device=device))
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        if kind == "prefix":
            self.x, self.wt, self.bias = mk(40, (L, B, D)), mk(41, (L, P * D, D)), mk(42, (L, P * D))
            self.out = torch.empty((L, B, P, D), dtype=torch.bfloat16, device=device)
            self.M, self.N, self.K = B, P * D, D
        else:
            self.x, self.wt, self.bias = mk(43, (L, B, 1, D)), mk(44, (L, 3 * D, D)), mk(45, (L, 3 * D))
            self.out = torch.empty((L, B, H, 1, hd), dtype=torch.bfloat16, device=device)
            self.M, self.N, self.K = B, 3 * D, D
            L = w.n_layers
            if kind == "qkv_token":
                self.cache = bt.LocalCache(self.cfg, device)
            else:
                self.cache = bt.BlockCache(self.cfg, device)
                self.len0 = torch.full((L, B), w.ctx_blocks - 1, dtype=torch.int32, device=device)
                self.cache.len.copy_(self.len0)
        self.launches_per_step = w.n_layers
        self.graph = None

    def step(self, s=0):
        for l in range(self.w.n_layers):
            i = s * self.w.n_layers + l
            if self.kind == "prefix":
                bt.bt_prefix_project(self.cfg, self.x[i], self.wt[i], self.bias[i], self.out[i], dev_status=self.status)
            elif self.kind == "qkv_token":
                bt.bt_local_qkv_project_append(self.cfg, self.cache, l, self.x[i], self.wt[i], self.bias[i], self.out[i],
                                               reset_first=True, dev_status=self.status)
            else:
                bt.bt_block_qkv_project_append(self.cfg, self.cache, l, self.x[i], self.wt[i], self.bias[i], self.out[i],
                                               dev_status=self.status)

    def rewind(self):
        if self.kind == "qkv_block":
            self.cache.len.copy_(self.len0, non_blocking=True)

    def capture(self):
        self.rewind()
        self.step()
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            for s in range(self.sets):
                self.rewind()
                self.step(s)

    def replay(self):
        """`sets` steps."""
        self.graph.replay()


class ProjectedTokenRun:
    """Token-decoder steps with the QKV projection in the path (sections 2.3 and 2.4 with the projections either
    side): per layer and step, the layer's input x [B,1,D] is projected, the epilogue writes the K and V rows
    into the local cache (reset at the first step of a block) and q goes to the attention call, which attends
    over the cache as it stands (nothing left to append).  Two library calls per layer and step; distinct
    weights per layer; step inputs rotate over a ring.  Prefix length 1: the block start is a one-row step too."""

    def __init__(self, w, device="cuda", fill=None, ring=8):
        assert w.prefix_len == 1
        self.w, self.ring = w, ring
        L, B, H, hd = w.n_layers, w.batch, w.heads, w.head_dim
        D = H * hd
        self.cfg = bt.make_config(B, H, hd, w.block_len, w.prefix_len, max(1, w.max_blocks), L)
        mk = fill if fill is not None else (lambda tid, sh: torch.zeros(sh, dtype=torch.bfloat16, device=device))
        self.cache = bt.LocalCache(self.cfg, device)
        self.x = mk(50, (ring, L, B, 1, D))
        self.x.mul_(1.0 / D ** 0.5)   # unit-variance q and k after the projection, as every attention input here
        self.wt, self.bias = mk(51, (L, 3 * D, D)), mk(52, (L, 3 * D))
        self.q = torch.empty((L, B, H, 1, hd), dtype=torch.bfloat16, device=device)
        self.out = torch.empty((L, B, H, 1, hd), dtype=torch.bfloat16, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.t = 0
        self.launches_per_step = 3 * L   # product, length update, attention

    def token_step(self):
        w = self.w
        first = self.t % w.block_len == 0
        r = self.t % self.ring
        for l in range(w.n_layers):
            bt.bt_local_qkv_project_append(self.cfg, self.cache, l, self.x[r, l], self.wt[l], self.bias[l], self.q[l],
                                           reset_first=first, dev_status=self.status)
            bt.bt_token_decode_attn(self.cfg, self.cache, l, self.q[l], None, None, self.out[l], n_q=1, dev_status=self.status)
        self.t += 1

    def capture(self, n_steps=None):
        n_steps = self.ring if n_steps is None else n_steps
        assert n_steps % self.w.block_len == 0 and self.t % self.w.block_len == 0
        for _ in range(self.w.block_len):
            self.token_step()   # anything lazy happens outside the capture; a whole block keeps the phase
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            for _ in range(n_steps):
                self.token_step()
        return n_steps

    def replay(self):
        self.graph.replay()
