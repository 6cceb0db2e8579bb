#!/usr/bin/env python
"""Benchmark of the renderer chunk-attention path on B200.

One step = one steady-state renderer chunk through the whole hot path on one GPU: for every denoising stage
(S = 4) and every layer (30): rotary embedding of Q/K, in-place publish of (K', V) into the stage's ring,
flash attention over [anchor | history | own chunk]; then Tail_H for the stage; plus the anchor publishes that
fall on that chunk (one anchor frame, all layers, every 4th chunk).  Workload: the Wan-1.3B-shaped 480p
configuration (second entry of the benchmark's config list).

    python bench.py [--gpus N] [--steps K] [--warmup W]            # this library
    python bench.py --impl reference [--steps K] [--warmup W]      # the CPU oracle as the reference arm

Prints ONE JSON line on rank 0.  With N > 1 (torchrun) every rank runs an independent replica of the same
stream on its own GPU ("replicas only": the path has no exchange step); value is the sum over ranks divided
by the slowest rank's time.
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
sys.path.insert(0, ROOT)

import torch  # noqa: E402

import ff_workloads as W  # noqa: E402

WORKLOAD = "wan1p3b_480p"
NOMINAL_BF16_TFLOPS = 2250.0
N_IO = 8                 # distinct resident Q/K/V sets cycled over the layer-calls (345 MB > the 126 MB L2)
CPU_SAMPLE_ROWS = 0      # query rows of one steady-state layer-call the oracle is timed on (0 = all of them)
# committed ncu summaries of the dominant kernel, by workload (each names the kernel source it was captured from)
ATTN_PROFILES = {"wan1p3b_480p": os.path.join(ROOT, "profiles", "attn_tcgen05_wan1p3b_480p.json"),
                 "wan1p3b_720p": os.path.join(ROOT, "profiles", "attn_pair_wan1p3b_720p.json")}


def blob_hash(paths) -> str:
    """One hash over the contents of the files (in the given order): sha1 of their git blob hashes."""
    import hashlib
    h = hashlib.sha1()
    for path in paths:
        data = open(os.path.join(ROOT, path), "rb").read()
        h.update(hashlib.sha1(b"blob %d\0" % len(data) + data).hexdigest().encode())
    return h.hexdigest()


def ncu_traffic(workload: str) -> dict:
    """DRAM bytes per attention launch from the committed ncu summary of this workload, with a flag that says
    whether the kernel's source has changed since that capture (then the figure describes an older kernel)."""
    path = ATTN_PROFILES.get(workload)
    if path is None or not os.path.exists(path):
        return dict(traffic=None, traffic_source="no ncu capture of this workload")
    prof = json.load(open(path))
    per_launch = prof["dram_bytes_read_per_launch"] + prof["dram_bytes_write_per_launch"]
    return dict(traffic=per_launch, traffic_source=os.path.relpath(path, ROOT), traffic_kernel=prof["kernel"],
                traffic_stale=blob_hash(prof["kernel_sources"]) != prof["kernel_sources_hash"],
                traffic_captured_on=prof.get("capture_case"),
                tensor_pipe_active_pct_in_capture=prof.get("sm_pipe_tensor_cycles_active_pct_elapsed"))


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(source="measured", burst=float(p["bf16_tflops"]), sustained=float(p["bf16_tflops_sustained"]),
                    hbm_gbs=float(p["hbm_gbs"]))
    return dict(source="fallback", burst=1590.0, sustained=1400.0, hbm_gbs=6650.0)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        busy = [c for c, p in zip(sm, pw) if p > 0.5 * max(pw)] or sm
        return dict(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), power_w_max=max(pw), samples=len(sm),
                    reasons=sorted(reasons))


def max_over_ranks(x: float, world: int, device) -> float:
    """Slowest rank's time: every rank contributes its device-timed milliseconds."""
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_rank: float, ms: float, world: int) -> float:
    """Replicas: every rank did flops_per_rank; the job took the slowest rank's ms."""
    return world * flops_per_rank / (ms * 1e-3) / 1e12


def attn_algorithmic_bytes(w: W.Workload) -> float:
    """HBM bytes one steady-state attention launch cannot avoid: rotated queries in, output out, every visible key
    and value row once (bf16)."""
    n_q = w.chunk_frames * w.tokens_per_frame
    return 2.0 * w.n_heads * w.head_dim * (2 * n_q + 2 * w.steady_n_kv())


def chunk_flops(w: W.Workload, i: int) -> float:
    """Exact attention flops of all S*Ly layer-calls of chunk i (only keys that are really visible)."""
    n_q = w.chunk_frames * w.tokens_per_frame
    n_kv = (len(W.visible_anchor_ids(w, i)) + min(i, w.history_chunks) * w.chunk_frames + w.chunk_frames) \
        * w.tokens_per_frame
    return w.flops_per_call(n_q, n_kv) * w.n_stages * w.n_layers


# ----------------------------------------------------------------------------------------------- CPU oracle leg

class OracleStream:
    """The CPU oracle, as it stands, walking a steady-state stream of one layer at the benchmark's shape: the
    anchor and the first H chunks are published up front; every timed step is the layer-call of the next chunk
    restricted to n_rows query rows (each row still sees all visible keys; the rotary embedding and publish of
    the whole chunk are part of the call)."""

    def __init__(self, w: W.Workload):
        from oracle import ff_oracle as O
        self.O, self.w = O, w
        self.orc = O.Oracle(1, w.n_heads, w.head_dim, w.grid_h, w.grid_w, w.chunk_frames, 1, w.history_chunks, 1,
                            dtype=O.BF16, rope_theta=w.rope_theta)
        k, v = W.anchor_kv(w, 0, 0, 0)
        assert self.orc.anchor_publish(0, W.anchor_frame_pos(w, 0), 0, k.float().numpy(), v.float().numpy()) == 0
        q, k, v = W.qkv(w, 0, 0, 0, 0)
        self.q, self.k, self.v = q.float().numpy(), k.float().numpy(), v.float().numpy()
        self.chunk = 0
        for _ in range(w.history_chunks):
            self.step(0)

    def step(self, n_rows: int):
        """Returns (TFLOP/s, seconds) of one layer-call on n_rows sampled rows (n_rows = 0: publish only)."""
        w, i = self.w, self.chunk
        n_q = w.chunk_frames * w.tokens_per_frame
        rows = None if n_rows >= n_q else [int(r * n_q / n_rows) for r in range(n_rows)]
        n_rows = min(n_rows, n_q)
        t0 = time.perf_counter()
        st, _ = self.orc.chunk_forward(0, 0, i, w.chunk_frames, i * w.chunk_frames, self.q, self.k, self.v, [0],
                                       rows=rows)
        dt = time.perf_counter() - t0
        assert st == 0 and self.orc.advance(0) == 0
        self.chunk += 1
        flops = 4.0 * n_rows * w.steady_n_kv() * w.head_dim * w.n_heads
        return flops / dt / 1e12, dt

    def threads(self) -> int:
        return self.O.num_threads()


def oracle_sample(w: W.Workload, n_rows: int):
    """One timed steady-state sample: (TFLOP/s, seconds, threads)."""
    s = OracleStream(w)
    v, dt = s.step(n_rows or w.chunk_frames * w.tokens_per_frame)
    return v, dt, s.threads()


def oracle_tiny_stream() -> dict:
    """The smallest configuration in full on the CPU oracle: every chunk, stage and layer-call of its stream."""
    from oracle import ff_oracle as O
    w = W.CONFIGS["tiny"]
    orc = O.Oracle(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
                   chunk_frames=w.chunk_frames, n_stages=w.n_stages, history_chunks=w.history_chunks,
                   n_anchor_slots=w.n_anchor_slots, dtype=O.BF16, rope_theta=w.rope_theta)
    inputs = {}
    for ev in W.trace(w):
        if ev.kind == "anchor":
            inputs[("a", ev.anchor_id)] = [tuple(t.float().numpy() for t in W.anchor_kv(w, 0, ev.anchor_id, l))
                                           for l in range(w.n_layers)]
        else:
            for stage in range(w.n_stages):
                for l in range(w.n_layers):
                    inputs[(ev.chunk, stage, l)] = tuple(t.float().numpy() for t in W.qkv(w, 0, ev.chunk, stage, l, ev.n_frames))
    t0 = time.perf_counter()
    flops = 0.0
    for ev in W.trace(w):
        if ev.kind == "anchor":
            for l in range(w.n_layers):
                k, v = inputs[("a", ev.anchor_id)][l]
                assert orc.anchor_publish(ev.slot, ev.frame_pos, l, k, v) == 0
            continue
        for stage in reversed(range(w.n_stages)):
            for l in range(w.n_layers):
                q, k, v = inputs[(ev.chunk, stage, l)]
                st, _ = orc.chunk_forward(stage, l, ev.chunk, ev.n_frames, ev.first_frame_pos, q, k, v, ev.anchor_slots)
                assert st == 0
            assert orc.advance(stage) == 0
        flops += chunk_flops(w, ev.chunk)
    dt = time.perf_counter() - t0
    return dict(workload="tiny", chunks=w.n_chunks, layer_calls=w.n_chunks * w.n_stages * w.n_layers, seconds=dt,
                tflops=flops / dt / 1e12)


def config_dict(w: W.Workload, world: int, name: str = WORKLOAD) -> dict:
    return dict(workload=name, n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim,
                tokens_per_frame=w.tokens_per_frame, chunk_frames=w.chunk_frames, n_stages=w.n_stages,
                history_chunks=w.history_chunks, visible_anchors=w.visible_anchors,
                n_q=w.chunk_frames * w.tokens_per_frame, n_kv=w.steady_n_kv(),
                layer_calls_per_step=w.n_stages * w.n_layers, parallelism=f"replicas x{world}",
                l2=(f"inputs larger than L2 ({N_IO} Q/K/V sets = "
                    f"{3 * N_IO * w.chunk_frames * w.tokens_per_frame * w.n_heads * w.head_dim * 2 / 1e6:.0f} MB cycled, "
                    f"on top of the ring)"))


def run_reference(args):
    """Reference arm: the CPU oracle on the host cores; each step is a bounded sample of the workload (one
    steady-state layer-call on 128 of its 4680 query rows)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = W.CONFIGS[WORKLOAD]
    n_rows = 128
    stream = OracleStream(w)
    for _ in range(args.warmup):
        stream.step(16)
    vals, secs = [], []
    for _ in range(args.steps):
        v, dt = stream.step(n_rows)
        vals.append(v); secs.append(dt)
    threads = stream.threads()
    value = sum(vals) / len(vals)
    sample = (f"{n_rows} of {w.chunk_frames * w.tokens_per_frame} query rows x {w.n_heads} heads of one steady-state "
              f"layer-call (N_kv={w.steady_n_kv()}) per step, rotary+publish of the whole chunk included")
    line = dict(impl="reference", metric="chunk_attn_tflops", value=value, unit="TFLOP/s", n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=1e3 * sum(secs) / len(secs), higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic", config=config_dict(w, args.gpus),
                cpu_baseline=dict(value=value, unit="TFLOP/s", cores=threads, kind="oracle", sample=sample),
                e2e=dict(value=value, unit="TFLOP/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- GPU arm

def measure_paper_budget(P, dev, local: int, steps: int = 3) -> dict:
    """Extra, outside the benchmark's metric: the same kernels at the paper's own context budget (W_ctx = 21
    latent positions).  Renderer: H = 5 history chunks and three anchors chosen by Gamma(i); planner: blocks of
    three anchor latents over Tail_6 of the clean bank, S denoising forwards plus the clean-endpoint forward."""
    out = {}
    for role, w0, calls_per_layer in (("renderer", W.PAPER_480P, None), ("planner", W.PAPER_480P_PLANNER, 5)):
        warm = w0.history_chunks + 1
        n_units = warm + steps
        w = W.scaled(w0, total_frames=(n_units + 1) * w0.chunk_frames,
                     max_frame_pos=(n_units + 2) * w0.chunk_frames * w0.frame_pos_stride + 64)
        cfg = P.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h,
                            grid_w=w.grid_w, chunk_frames=w.chunk_frames, n_stages=w.n_stages,
                            history_chunks=w.history_chunks, n_anchor_slots=w.n_anchor_slots,
                            max_visible_anchors=w.visible_anchors, dtype=P.FF_BF16, attn_impl=P.FF_ATTN_AUTO,
                            max_frame_pos=w.max_frame_pos, rope_theta=w.rope_theta, device=local,
                            frame_pos_stride=w.frame_pos_stride, allow_republish=int(w.allow_republish))
        nbytes = P.ff_cache_query_bytes(cfg)
        arena = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        cache = P.Cache(cfg, arena.data_ptr(), nbytes)
        stream = torch.cuda.current_stream().cuda_stream
        sets = []
        for sidx in range(N_IO):
            q, k, v = W.qkv(w, 1, sidx, 0, 0)
            sets.append((q.to(dev), k.to(dev), v.to(dev), torch.empty_like(q, device=dev)))
        io = P.make_io([(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr()) for q, k, v, o in sets])
        ak, av = (t.to(dev) for t in W.anchor_kv(w, 1, 0, 0))
        published = set()

        def unit(i):
            ids = W.visible_anchor_ids(w, i)
            for m in ids:
                if m not in published:
                    published.add(m)
                    for l in range(w.n_layers):
                        assert cache.ff_anchor_publish(W.anchor_slot(w, m), W.anchor_frame_pos(w, m), l, ak.data_ptr(),
                                                       av.data_ptr(), stream) == 0
            slots = [W.anchor_slot(w, m) for m in ids]
            pos = i * w.chunk_frames * w.frame_pos_stride
            if calls_per_layer is None:
                assert cache.ff_sched_run_chunk(i, w.chunk_frames, pos, slots, io, stream) == 0
            else:
                for f in range(calls_per_layer):
                    for l in range(w.n_layers):
                        q, k, v, o = sets[(f * w.n_layers + l) % N_IO]
                        assert cache.ff_chunk_forward_attn(0, l, i, w.chunk_frames, pos, q.data_ptr(), k.data_ptr(),
                                                           v.data_ptr(), slots, o.data_ptr(), stream) == 0
                assert cache.ff_cache_advance(0) == 0

        for i in range(warm):
            unit(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(warm, warm + steps):
            unit(i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        calls = w.n_stages * w.n_layers * (calls_per_layer or 1)
        flops = w.flops_per_call() * calls
        out[role] = dict(workload=w0.name, n_q=w.chunk_frames * w.tokens_per_frame, n_kv=w.steady_n_kv(),
                         layer_calls_per_step=calls, steps=steps, ms_per_step=ms, tflops=flops / (ms * 1e-3) / 1e12)
        cache.close()
        del arena, sets
        torch.cuda.empty_cache()
    return out


def measure_wavefront(P, dev, local: int, workload: str, steps: int) -> dict:
    """Extra: the same chunks in wavefront order (Alg. 1 Phase B on one device).  Round n holds the nodes
    (chunk n - r, stage S - r), r = 0..S-1, which are independent; per layer they share one attention launch.  In
    steady state a round does exactly the work of one chunk-major step (S stages x all layers) and completes one
    chunk, so ms per round and TFLOP/s compare directly with the headline."""
    base = W.CONFIGS[workload]
    S, H = base.n_stages, base.history_chunks
    warm = (S - 1) + (H + 1) + 2
    n_rounds = warm + steps
    w = W.scaled(base, total_frames=(n_rounds + 2) * base.chunk_frames, clip_anchor_pos=False,
                 max_frame_pos=(n_rounds + 12) * base.chunk_frames + 16)
    cfg = P.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
                        chunk_frames=w.chunk_frames, n_stages=w.n_stages, history_chunks=w.history_chunks,
                        n_anchor_slots=w.n_anchor_slots, max_visible_anchors=w.visible_anchors, dtype=P.FF_BF16,
                        attn_impl=P.FF_ATTN_AUTO, max_frame_pos=w.max_frame_pos, rope_theta=w.rope_theta,
                        device=local)
    nbytes = P.ff_cache_query_bytes(cfg)
    arena = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    cache = P.Cache(cfg, arena.data_ptr(), nbytes)
    stream = torch.cuda.current_stream().cuda_stream
    sets = []
    for sidx in range(N_IO):
        q, k, v = W.qkv(w, 3, sidx, 0, 0)
        sets.append((q.to(dev), k.to(dev), v.to(dev), torch.empty_like(q, device=dev)))
    # node r of a round takes the sets r, r + S, ... in turn over the layers: distinct buffers inside a launch
    ios = [P.make_io([(sets[(r + S * l) % N_IO][0].data_ptr(), sets[(r + S * l) % N_IO][1].data_ptr(),
                       sets[(r + S * l) % N_IO][2].data_ptr(), sets[(r + S * l) % N_IO][3].data_ptr())
                      for l in range(w.n_layers)]) for r in range(S)]
    ak, av = (t.to(dev) for t in W.anchor_kv(w, 3, 0, 0))
    published = set()

    def run_round(n):
        if n >= 0:
            for m in W.visible_anchor_ids(w, n):
                if m not in published:
                    published.add(m)
                    for l in range(w.n_layers):
                        assert cache.ff_anchor_publish(W.anchor_slot(w, m), W.anchor_frame_pos(w, m), l, ak.data_ptr(),
                                                       av.data_ptr(), stream) == 0
        nodes = []
        for r in range(S):
            i = n - r
            if i < 0:
                continue
            nodes.append(dict(stage=S - 1 - r, chunk_index=i, n_frames=w.chunk_frames, first_frame_pos=i * w.chunk_frames,
                              anchor_slots=[W.anchor_slot(w, m) for m in W.visible_anchor_ids(w, i)], io=ios[r]))
        assert cache.ff_sched_run_round(nodes, stream) == 0

    for n in range(warm):
        run_round(n)
    torch.cuda.synchronize()
    c0 = cache.ff_cache_counters()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    marks[0].record()
    flops = 0.0
    for j in range(steps):
        n = warm + j
        run_round(n)
        marks[j + 1].record()
        flops += sum(chunk_flops(w, n - r) for r in range(S)) / S
    torch.cuda.synchronize()
    c1 = cache.ff_cache_counters()
    st, word = cache.ff_cache_status(stream)
    assert st == 0 and word == 0, (st, hex(word))
    ms = marks[0].elapsed_time(marks[steps])
    per = [marks[j].elapsed_time(marks[j + 1]) for j in range(steps)]
    out = dict(workload=workload, rounds=steps, nodes_per_round=S, layer_calls_per_round=S * w.n_layers,
               ms_per_round=ms / steps, ms_per_round_best=min(per), tflops=flops / (ms * 1e-3) / 1e12,
               chunks_per_s=steps / (ms * 1e-3), gpu_launches=c1["kernel_launches"] - c0["kernel_launches"])
    cache.close()
    del arena, sets
    torch.cuda.empty_cache()
    return out


def measure_clip_at_once(P, dev, local: int, group: int = 27) -> dict:
    """Extra: one stage of a whole 81-latent clip at the paper's budget (H = 5, Gamma windows, 27 chunks) in the
    clip-at-once form: `group` consecutive chunks of the stage per batched launch under the chunk-wise causal
    mask (bank with H + group slots), all layers.  group = 27 is the whole clip in ONE attention launch per
    layer."""
    w = W.scaled(W.PAPER_480P, n_stages=1, n_anchor_slots=9)
    N = w.n_chunks
    cfg = P.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
                        chunk_frames=w.chunk_frames, n_stages=1, history_chunks=w.history_chunks,
                        n_anchor_slots=w.n_anchor_slots, max_visible_anchors=w.visible_anchors, dtype=P.FF_BF16,
                        attn_impl=P.FF_ATTN_AUTO, max_frame_pos=w.max_frame_pos, rope_theta=w.rope_theta,
                        device=local, ring_slots=w.history_chunks + group, max_batch=group)
    nbytes = P.ff_cache_query_bytes(cfg)
    arena = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    cache = P.Cache(cfg, arena.data_ptr(), nbytes)
    stream = torch.cuda.current_stream().cuda_stream
    sets = []
    for sidx in range(max(N_IO, group)):
        q, k, v = W.qkv(w, 4, sidx, 0, 0)
        sets.append((q.to(dev), k.to(dev), v.to(dev), torch.empty_like(q, device=dev)))
    ios = [P.make_io([(sets[(r + group * l) % len(sets)][0].data_ptr(), sets[(r + group * l) % len(sets)][1].data_ptr(),
                       sets[(r + group * l) % len(sets)][2].data_ptr(), sets[(r + group * l) % len(sets)][3].data_ptr())
                      for l in range(w.n_layers)]) for r in range(group)]
    ak, av = (t.to(dev) for t in W.anchor_kv(w, 4, 0, 0))

    def clip(timed):
        assert cache.ff_cache_reset() == 0
        for m in range(9):
            for l in range(w.n_layers):
                assert cache.ff_anchor_publish(W.anchor_slot(w, m), W.anchor_frame_pos(w, m), l, ak.data_ptr(),
                                               av.data_ptr(), stream) == 0
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i0 in range(0, N, group):
            nodes = [dict(stage=0, chunk_index=i, n_frames=w.chunk_frames_of(i), first_frame_pos=i * w.chunk_frames,
                          anchor_slots=[W.anchor_slot(w, m) for m in W.visible_anchor_ids(w, i)], io=ios[i - i0])
                     for i in range(i0, min(i0 + group, N))]
            assert cache.ff_sched_run_round(nodes, stream) == 0
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    clip(False)
    ms = min(clip(True), clip(True))
    flops = sum(chunk_flops(w, i) for i in range(N))
    st, word = cache.ff_cache_status(stream)
    assert st == 0 and word == 0, (st, hex(word))
    out = dict(workload=w.name + ", one stage", chunks=N, group=group, layer_calls=N * w.n_layers, ms_per_clip_stage=ms,
               tflops=flops / (ms * 1e-3) / 1e12)
    cache.close()
    del arena, sets
    torch.cuda.empty_cache()
    return out


def measure_peaked_logits(P, dev, local: int, workload: str, steps: int, logit_gain: float = 8.0) -> dict:
    """Extra: the headline step on inputs whose logits are `logit_gain` times larger (peaked softmax).  The
    attention kernel raises a row's reference maximum lazily and rescales its accumulator when it does, so its
    speed depends on the data; the headline's RMS-normalised inputs hardly ever trigger that path, these do."""
    base = W.CONFIGS[workload]
    warm = base.history_chunks + 2
    w = W.scaled(base, total_frames=(warm + steps + 2) * base.chunk_frames, clip_anchor_pos=False,
                 max_frame_pos=(warm + steps + 12) * base.chunk_frames + 16)
    cfg = P.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
                        chunk_frames=w.chunk_frames, n_stages=w.n_stages, history_chunks=w.history_chunks,
                        n_anchor_slots=w.n_anchor_slots, max_visible_anchors=w.visible_anchors, dtype=P.FF_BF16,
                        attn_impl=P.FF_ATTN_AUTO, max_frame_pos=w.max_frame_pos, rope_theta=w.rope_theta,
                        device=local)
    nbytes = P.ff_cache_query_bytes(cfg)
    arena = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    cache = P.Cache(cfg, arena.data_ptr(), nbytes)
    stream = torch.cuda.current_stream().cuda_stream
    sets = []
    for sidx in range(N_IO):
        q, k, v = W.qkv(w, 5, sidx, 0, 0, logit_gain=logit_gain)
        sets.append((q.to(dev), k.to(dev), v.to(dev), torch.empty_like(q, device=dev)))
    io = P.make_io([(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr()) for q, k, v, o in sets])
    ak, av = (t.to(dev) for t in W.anchor_kv(w, 5, 0, 0))
    published = set()

    def step(i):
        ids = W.visible_anchor_ids(w, i)
        for m in ids:
            if m not in published:
                published.add(m)
                for l in range(w.n_layers):
                    assert cache.ff_anchor_publish(W.anchor_slot(w, m), W.anchor_frame_pos(w, m), l, ak.data_ptr(),
                                                   av.data_ptr(), stream) == 0
        assert cache.ff_sched_run_chunk(i, w.chunk_frames, i * w.chunk_frames, [W.anchor_slot(w, m) for m in ids], io,
                                        stream) == 0

    for i in range(warm):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    flops = 0.0
    for i in range(warm, warm + steps):
        step(i)
        flops += chunk_flops(w, i)
    e1.record()
    torch.cuda.synchronize()
    st, word = cache.ff_cache_status(stream)
    assert st == 0 and word == 0, (st, hex(word))
    ms = e0.elapsed_time(e1)
    # how peaked: share of a row's probability mass on its largest key, for a few rows of one head (diagnostic)
    q, k = sets[0][0][:64, 0].float(), torch.cat([s_[1][:, 0].float() for s_ in sets[:3]])
    p = torch.softmax(q @ k.T / w.head_dim ** 0.5, dim=-1)
    out = dict(workload=workload, logit_gain=logit_gain, steps=steps, ms_per_step=ms / steps,
               tflops=flops / (ms * 1e-3) / 1e12, chunks_per_s=steps / (ms * 1e-3),
               mean_top1_probability_unrotated_sample=float(p.max(dim=-1).values.mean()))
    cache.close()
    del arena, sets
    torch.cuda.empty_cache()
    return out


def measure_adjacent_steps(P, dev, local: int, hbm_peak_gbs: float) -> dict:
    """Extra, outside the benchmark's metric: the two steps next to the path.  (1) The publish pass with the q/k
    normalisation fused in, against the plain one, on the headline shape (4 layers are enough: the pass does not
    depend on the layer count).  (2) The Euler update after a forward at a chunk's latent size and at a size far
    beyond L2, where it is bound by HBM."""
    out = {}
    base = W.scaled(W.CONFIGS[WORKLOAD], n_layers=4, n_stages=1)
    n_units = base.history_chunks + 4
    w = W.scaled(base, total_frames=(n_units + 1) * base.chunk_frames, clip_anchor_pos=False,
                 max_frame_pos=(n_units + 8) * base.chunk_frames + 16)
    stream = torch.cuda.current_stream().cuda_stream
    for label, norm in (("publish_plain", 0), ("publish_with_qk_norm", 1)):
        cfg = P.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h,
                            grid_w=w.grid_w, chunk_frames=w.chunk_frames, n_stages=w.n_stages,
                            history_chunks=w.history_chunks, n_anchor_slots=w.n_anchor_slots,
                            max_visible_anchors=w.visible_anchors, dtype=P.FF_BF16, attn_impl=P.FF_ATTN_AUTO,
                            max_frame_pos=w.max_frame_pos, rope_theta=w.rope_theta, device=local, qk_norm=norm)
        nbytes = P.ff_cache_query_bytes(cfg)
        arena = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        cache = P.Cache(cfg, arena.data_ptr(), nbytes)
        sets = []
        for sidx in range(N_IO):
            q, k, v = W.qkv(w, 2, sidx, 0, 0, pre_normalised=not norm)
            sets.append((q.to(dev), k.to(dev), v.to(dev), torch.empty_like(q, device=dev)))
        io = P.make_io([(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr()) for q, k, v, o in sets])
        ak, av = (t.to(dev) for t in W.anchor_kv(w, 2, 0, 0, pre_normalised=not norm))
        published = set()

        def unit(i):
            ids = W.visible_anchor_ids(w, i)
            for m in ids:
                if m not in published:
                    published.add(m)
                    for l in range(w.n_layers):
                        assert cache.ff_anchor_publish(W.anchor_slot(w, m), W.anchor_frame_pos(w, m), l, ak.data_ptr(),
                                                       av.data_ptr(), stream) == 0
            assert cache.ff_sched_run_chunk(i, w.chunk_frames, i * w.chunk_frames, [W.anchor_slot(w, m) for m in ids],
                                            io, stream) == 0

        for i in range(n_units - 3):
            unit(i)
        assert cache.ff_cache_profile_begin(3 * w.n_layers) == 0
        for i in range(n_units - 3, n_units):
            unit(i)
        prof = cache.ff_cache_profile_end(stream)
        ms = prof["publish_ms"] / max(prof["publish_launches"], 1)
        nbytes_call = 6 * w.chunk_frames * w.tokens_per_frame * w.n_heads * w.head_dim * 2
        out[label] = dict(ms_per_launch=ms, gbs=nbytes_call / (ms * 1e-3) / 1e9,
                          frac_of_hbm_peak=nbytes_call / (ms * 1e-3) / 1e9 / hbm_peak_gbs, launches=prof["publish_launches"])
        cache.close()
        del arena, sets
        torch.cuda.empty_cache()
    # Euler update: fp32 latent, bf16 velocity (4 + 2 bytes read, 4 written per element)
    for label, n in (("euler_chunk_latent", 3 * 16 * 60 * 104), ("euler_hbm_bound", 1 << 28)):
        x = torch.zeros(n, dtype=torch.float32, device=dev)
        v = torch.ones(n, dtype=torch.bfloat16, device=dev)
        o = torch.empty_like(x)
        reps = 20
        for _ in range(3):
            assert P.ff_euler_step(x.data_ptr(), v.data_ptr(), 1.0, 0.9375, n, P.FF_F32, P.FF_BF16, o.data_ptr(), stream) == 0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            assert P.ff_euler_step(x.data_ptr(), v.data_ptr(), 1.0, 0.9375, n, P.FF_F32, P.FF_BF16, o.data_ptr(), stream) == 0
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        out[label] = dict(n=n, ms_per_launch=ms, gbs=10.0 * n / (ms * 1e-3) / 1e9,
                          frac_of_hbm_peak=10.0 * n / (ms * 1e-3) / 1e9 / hbm_peak_gbs)
        del x, v, o
        torch.cuda.empty_cache()
    return out


def pipeline_run(P, base: W.Workload, world: int, rank: int, steps: int, warmup: int, device_index, group=None) -> dict:
    """Stage-per-rank renderer wavefront (Alg. 1 Phase B): `world` ranks, rank r owns the S / world denoising stages
    r * S/world .. (r+1) * S/world - 1 counted from the noisiest, each in a cache of its own on its own device; a
    chunk's latent is handed from rank to rank point to point (torch.distributed isend / recv), the banks never
    move.  world = 1 is the chunk-major order on one device.  Runs `warmup` chunks untimed, then times `steps`
    chunks from a barrier until this rank has finished its last one (pipeline fill and drain included).
    device_index None = bookkeeping-only caches and CPU latents: the same code path without a GPU (tests)."""
    import torch.distributed as dist
    from paper_2609_32540_b200 import wavefront as Wf
    S = base.n_stages
    assert S % world == 0, "the ranks must share the denoising stages equally"
    n_local = S // world
    dry = device_index is None
    n_total = warmup + steps
    w = W.scaled(base, n_stages=n_local, total_frames=(n_total + 2) * base.chunk_frames, clip_anchor_pos=False,
                 max_frame_pos=(n_total + 12) * base.chunk_frames + 16,
                 n_anchor_slots=max(base.n_anchor_slots, 2 * base.visible_anchors + 1))
    dev = torch.device("cpu") if dry else torch.device(f"cuda:{device_index}")
    cfg = P.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
                        chunk_frames=w.chunk_frames, n_stages=n_local, history_chunks=w.history_chunks,
                        n_anchor_slots=w.n_anchor_slots, max_visible_anchors=w.visible_anchors, dtype=P.FF_BF16,
                        attn_impl=P.FF_ATTN_AUTO, max_frame_pos=w.max_frame_pos, rope_theta=w.rope_theta,
                        device=P.FF_DEVICE_NONE if dry else device_index)
    if dry:
        arena, cache, stream = None, P.Cache(cfg, None, 0), 0
        io = P.make_io([(16, 16, 16, 16)] * w.n_layers)
        ak_ptr = av_ptr = 16
    else:
        nbytes = P.ff_cache_query_bytes(cfg)
        arena = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        cache = P.Cache(cfg, arena.data_ptr(), nbytes)
        stream = torch.cuda.current_stream().cuda_stream
        sets = []
        for sidx in range(N_IO):
            q, k, v = W.qkv(w, 6, sidx, rank, 0)
            sets.append((q.to(dev), k.to(dev), v.to(dev), torch.empty_like(q, device=dev)))
        io = P.make_io([(sets[l % N_IO][0].data_ptr(), sets[l % N_IO][1].data_ptr(), sets[l % N_IO][2].data_ptr(),
                         sets[l % N_IO][3].data_ptr()) for l in range(w.n_layers)])
        ak, av = (t.to(dev) for t in W.anchor_kv(w, 6, 0, 0))
        ak_ptr, av_ptr = ak.data_ptr(), av.data_ptr()
    # the chunk's latent: 16 channels on a grid twice as fine as the token grid, float32; the velocity stands in
    # for the forward's prediction
    n_lat = w.chunk_frames * 16 * (2 * w.grid_h) * (2 * w.grid_w)
    like = torch.zeros(n_lat, dtype=torch.float32, device=dev)
    velocity = torch.ones(n_lat, dtype=torch.float32 if dry else torch.bfloat16, device=dev)
    levels = [(P.ff_plan_sigma(S - rank * n_local - j, S), P.ff_plan_sigma(S - rank * n_local - j - 1, S))
              for j in range(n_local)]
    stages = Wf.RendererStages(cache, P.binding, levels, io, velocity, stream, dry)
    published = set()

    def run_node(i, x):
        ids = W.visible_anchor_ids(w, i)
        for m in ids:       # every rank keeps its own copy of the clean anchor bank
            if m not in published:
                published.add(m)
                for l in range(w.n_layers):
                    st = cache.ff_anchor_publish(W.anchor_slot(w, m), W.anchor_frame_pos(w, m), l, ak_ptr, av_ptr, stream)
                    assert st == 0, st
        return stages.run_node(i, w.chunk_frames, i * w.chunk_frames, [W.anchor_slot(w, m) for m in ids], x)

    delivered = []
    noise = torch.full_like(like, 1.0)

    def make_rank(n_chunks, first):
        return Wf.StageRank(rank, world, n_chunks, like, obtain=(lambda i: noise.clone()) if rank == 0 else None,
                            run_node=run_node, deliver=lambda i, x: delivered.append(i), group=group, first_chunk=first)

    def barrier():
        if not dry:
            torch.cuda.synchronize()
        if world > 1:
            dist.barrier(group=group)

    make_rank(warmup, 0).run()
    barrier()
    c0 = cache.ff_cache_counters()
    t0 = time.perf_counter()
    if not dry:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
    stats = make_rank(steps, warmup).run()
    if not dry:
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
    else:
        ms = 1e3 * (time.perf_counter() - t0)
    c1 = cache.ff_cache_counters()
    st, word = cache.ff_cache_status(stream)
    assert st == 0 and word == 0, (st, hex(word))
    flops_rank = sum(chunk_flops(w, warmup + j) for j in range(steps))     # this rank's stages only
    res = dict(rank=rank, ms=ms, chunks=stats.chunks, sent=stats.sent, received=stats.received,
               layer_calls=c1["layer_calls"] - c0["layer_calls"], advances=c1["advances"] - c0["advances"],
               gpu_launches=c1["kernel_launches"] - c0["kernel_launches"], delivered=list(delivered),
               flops=flops_rank, stages_per_rank=n_local, latent_bytes=n_lat * 4, n_q=w.chunk_frames * w.tokens_per_frame,
               n_kv=w.steady_n_kv())
    cache.close()
    return res


def run_wavefront_mode(args):
    """bench.py --mode wavefront: the stage-per-GPU pipeline on --gpus ranks (torchrun), one JSON line from rank 0."""
    import torch.distributed as dist
    import paper_2609_32540_b200 as P

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    base = W.CONFIGS[args.workload]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    res = pipeline_run(P, base, world, rank, args.steps, max(args.warmup, base.history_chunks + 2), local)
    clocks = sampler.stop() if rank == 0 else {}
    ms = max_over_ranks(res["ms"], world, dev)
    flops = res["flops"]
    launches = res["gpu_launches"]
    if world > 1:
        t = torch.tensor([flops, float(launches)], device=dev, dtype=torch.float64)
        dist.all_reduce(t)
        flops, launches = float(t[0].item()), int(t[1].item())
    if rank == 0:
        peaks = read_peaks()
        value = flops / (ms * 1e-3) / 1e12
        cfg = config_dict(base, world, args.workload)
        cfg["parallelism"] = f"stage pipeline x{world} ({res['stages_per_rank']} denoising stage(s) per rank)"
        line = dict(metric="chunk_attn_tflops", value=value, unit="TFLOP/s", n_gpus=world, steps=args.steps,
                    warmup=max(args.warmup, base.history_chunks + 2), ms_per_step=ms / args.steps, higher_is_better=True,
                    scaling="pipeline", vs_baseline=None, dtype="bf16", data="synthetic", mode="wavefront", config=cfg,
                    chunks_per_s=args.steps / (ms * 1e-3), clocks=clocks, gpu_launches=launches,
                    pct_of_measured_bf16_peak=100.0 * value / world / peaks["burst"],
                    latent_bytes_per_hop=res["latent_bytes"],
                    note=("timed from a barrier until the slowest rank has finished its last chunk: pipeline fill and "
                          "drain included; with one rank this is the chunk-major order plus the Euler updates"))
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_gpu(args):
    import torch.distributed as dist
    import paper_2609_32540_b200 as P

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    base = W.CONFIGS[args.workload]
    if args.layers:
        base = W.scaled(base, n_layers=args.layers)   # reduced profiling case, never a headline number
    K, Wm = args.steps, max(args.warmup, 3)
    n_total = Wm + K + args.e2e_steps + 1 + K
    w = W.scaled(base, total_frames=(n_total + 4) * base.chunk_frames, clip_anchor_pos=False,
                 max_frame_pos=max((n_total + 12) * base.chunk_frames + 16, base.total_frames + 16 if args.stream else 0))
    cfg = P.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
                        chunk_frames=w.chunk_frames, n_stages=w.n_stages, history_chunks=w.history_chunks,
                        n_anchor_slots=w.n_anchor_slots, max_visible_anchors=w.visible_anchors, dtype=P.FF_BF16,
                        attn_impl=P.FF_ATTN_AUTO, max_frame_pos=w.max_frame_pos, rope_theta=w.rope_theta,
                        device=local)
    nbytes = P.ff_cache_query_bytes(cfg)
    arena = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    cache = P.Cache(cfg, arena.data_ptr(), nbytes)
    stream = torch.cuda.current_stream().cuda_stream

    # resident inputs: N_IO distinct seeded Q/K/V sets (larger than L2 together), one output buffer per set
    sets = []
    for s in range(N_IO):
        q, k, v = W.qkv(w, 0, s, 0, 0)
        sets.append((q.to(dev), k.to(dev), v.to(dev), torch.empty_like(q, device=dev)))
    io = P.make_io([(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr()) for q, k, v, o in sets])
    ak, av = W.anchor_kv(w, 0, 0, 0)
    ak, av = ak.to(dev), av.to(dev)
    # pinned host buffers for the end-to-end leg (two sets)
    hsets = []
    for s in range(2):
        q, k, v = W.qkv(w, 0, 100 + s, 0, 0)
        hsets.append((q.pin_memory(), k.pin_memory(), v.pin_memory(), torch.empty_like(q).pin_memory()))
    hio = P.make_io([(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr()) for q, k, v, o in hsets])

    published = set()

    def step(i, host=False):
        """Chunk i through the whole path."""
        ids = W.visible_anchor_ids(w, i)
        for m in ids:
            if m not in published:   # first chunk that reads anchor m
                published.add(m)
                for l in range(w.n_layers):
                    st = cache.ff_anchor_publish(W.anchor_slot(w, m), W.anchor_frame_pos(w, m), l, ak.data_ptr(),
                                                 av.data_ptr(), stream)
                    assert st == 0, st
        slots = [W.anchor_slot(w, m) for m in ids]
        fn = cache.ff_sched_run_chunk_host if host else cache.ff_sched_run_chunk
        st = fn(i, w.chunk_frames, i * w.chunk_frames, slots, hio if host else io, stream)
        assert st == 0, st

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    chunk = 0
    for _ in range(Wm):
        step(chunk); chunk += 1
    # ---- timed region 1: K steps, inputs resident in HBM
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    c0 = cache.ff_cache_counters()
    flops = sum(chunk_flops(w, chunk + j) for j in range(K))
    barrier()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    marks[0].record()
    for j in range(K):
        step(chunk); chunk += 1
        marks[j + 1].record()
    barrier()
    e0, e1 = marks[0], marks[K]
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    per_step = [marks[j].elapsed_time(marks[j + 1]) for j in range(K)]
    clocks = sampler.stop() if rank == 0 else {}
    c1 = cache.ff_cache_counters()
    launches = c1["kernel_launches"] - c0["kernel_launches"]
    choice = cache.ff_cache_kernel_choice()
    attn_kernel = (f"attn_pair_kernel<false> on CTA pairs" if choice["cta_pair"] > choice["one_cta"]
                   else f"attn_tcgen05_kernel<{w.head_dim}, false, false>") + f" (+ attn_combine_kernel<{w.head_dim}, false>)"
    st, word = cache.ff_cache_status(stream)
    assert st == 0 and word == 0, (st, hex(word))

    # ---- timed region 2: the same K steps with per-kernel CUDA events (roofline of the dominant kernel)
    calls = K * w.n_stages * w.n_layers
    assert cache.ff_cache_profile_begin(calls) == 0
    barrier()
    for _ in range(K):
        step(chunk); chunk += 1
    prof = cache.ff_cache_profile_end(stream)
    attn_flops_per_launch = w.flops_per_call()
    # per layer-call: one publish launch, and one attention launch followed (when pairs were split) by a merge launch
    attn_ms = prof["attn_ms"] / calls
    publish_ms = prof["publish_ms"] / calls
    attn_tflops = attn_flops_per_launch / (attn_ms * 1e-3) / 1e12
    elem = 2
    publish_bytes = 6 * w.chunk_frames * w.tokens_per_frame * w.n_heads * w.head_dim * elem  # read q,k,v; write q',k',v
    publish_gbs = publish_bytes / (publish_ms * 1e-3) / 1e9

    # ---- end-to-end: host buffers, copies inside the timed region
    e2e_ms, e2e_flops = None, 0.0
    if args.e2e_steps > 0:
        step(chunk, host=True); chunk += 1
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        e2e_flops = sum(chunk_flops(w, chunk + j) for j in range(args.e2e_steps))
        for _ in range(args.e2e_steps):
            step(chunk, host=True); chunk += 1
        g1.record()
        barrier()
        e2e_ms = max_over_ranks(g0.elapsed_time(g1), world, dev)
    call_bytes = w.chunk_frames * w.tokens_per_frame * w.n_heads * w.head_dim * elem
    n_calls = w.n_stages * w.n_layers

    # ---- optional: the workload's whole stream from empty banks (warm-up chunks and anchor publishes included)
    stream_res = None
    if args.stream:
        assert cache.ff_cache_reset() == 0
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        seen, stream_flops = set(), 0.0
        for i in range(base.n_chunks):
            ids = W.visible_anchor_ids(base, i)
            for m in ids:
                if m not in seen:
                    seen.add(m)
                    for l in range(base.n_layers):
                        assert cache.ff_anchor_publish(W.anchor_slot(base, m), W.anchor_frame_pos(base, m), l,
                                                       ak.data_ptr(), av.data_ptr(), stream) == 0
            assert cache.ff_sched_run_chunk(i, base.chunk_frames_of(i), i * base.chunk_frames,
                                            [W.anchor_slot(base, m) for m in ids], io, stream) == 0
            stream_flops += chunk_flops(base, i) * base.chunk_frames_of(i) / base.chunk_frames
        s1.record()
        barrier()
        stream_ms = max_over_ranks(s0.elapsed_time(s1), world, dev)
        st, word = cache.ff_cache_status(stream)
        assert st == 0 and word == 0, (st, hex(word))
        stream_res = dict(chunks=base.n_chunks, frames=base.total_frames, anchor_frames=len(seen), seconds=stream_ms * 1e-3,
                          tflops=whole_job_tflops(stream_flops, stream_ms, world),
                          chunks_per_s=world * base.n_chunks / (stream_ms * 1e-3))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks = read_peaks()
    value = whole_job_tflops(flops, ms, world)
    cpu_v, cpu_dt, cpu_threads = (oracle_sample(base, CPU_SAMPLE_ROWS)
                                  if world == 1 and not args.skip_cpu and args.workload == WORKLOAD
                                  else (None, None, None))
    line = dict(
        metric="chunk_attn_tflops", value=value, unit="TFLOP/s", n_gpus=world, steps=K, warmup=Wm,
        ms_per_step=ms / K, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
        config=config_dict(w, world, args.workload),
        chunks_per_s=world * K / (ms * 1e-3),
        ms_per_step_best=min(per_step), ms_per_step_std=(statistics.pstdev(per_step) if K > 1 else 0.0),
        pct_of_measured_bf16_peak=100.0 * value / world / peaks["burst"],
        pct_of_nominal_bf16_peak=100.0 * value / world / NOMINAL_BF16_TFLOPS,
        clocks=clocks,
        e2e=(dict(value=whole_job_tflops(e2e_flops, e2e_ms, world), unit="TFLOP/s",
                  h2d_bytes_per_step=3 * call_bytes * n_calls, d2h_bytes_per_step=call_bytes * n_calls,
                  steps=args.e2e_steps, ms_per_step=e2e_ms / args.e2e_steps) if e2e_ms else None),
        gpu_launches=launches,
        roofline=dict(bound="tensor", kernel=attn_kernel, kernel_launches_by_choice=choice,
                      achieved=attn_tflops, peak=peaks["sustained"],
                      unit="TFLOP/s", frac=attn_tflops / peaks["sustained"], frac_of_burst_peak=attn_tflops / peaks["burst"],
                      peak_source=f"{peaks['source']} bf16 GEMM, sustained (kernel timed inside a long step)",
                      ms_per_launch=attn_ms, layer_calls_timed=calls, launches_timed=prof["attn_launches"],
                      flops_per_launch=attn_flops_per_launch, **ncu_traffic(args.workload),
                      algorithmic_bytes_per_launch=attn_algorithmic_bytes(w),
                      publish=dict(bound="hbm", achieved=publish_gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                                   frac=publish_gbs / peaks["hbm_gbs"], ms_per_launch=publish_ms,
                                   bytes_per_launch=publish_bytes)),
    )
    if stream_res is not None:
        line["whole_stream"] = stream_res
    if args.workload != WORKLOAD:
        line["note"] = "not the benchmark's headline configuration (that is the default workload)"
    if not args.layers and world == 1 and not args.skip_extra and args.workload == WORKLOAD:
        cache.close()
        del arena
        torch.cuda.empty_cache()
        line["paper_budget"] = measure_paper_budget(P, dev, local)
        line["adjacent_steps"] = measure_adjacent_steps(P, dev, local, peaks["hbm_gbs"])
        line["wavefront_rounds"] = measure_wavefront(P, dev, local, args.workload, K)
        line["peaked_logits"] = measure_peaked_logits(P, dev, local, args.workload, K)
        line["clip_at_once"] = measure_clip_at_once(P, dev, local, group=27)
    if args.layers:
        line["profile_case"] = f"reduced to {args.layers} layers: not a benchmark result"
    if cpu_v is not None:
        line["cpu_baseline"] = dict(
            value=cpu_v, unit="TFLOP/s", cores=cpu_threads, kind="oracle", seconds=cpu_dt,
            sample=(f"{CPU_SAMPLE_ROWS or w.chunk_frames * w.tokens_per_frame} of {w.chunk_frames * w.tokens_per_frame} "
                    f"query rows x {w.n_heads} heads of one steady-state layer-call (N_kv={w.steady_n_kv()}), rotary+publish "
                    f"of the whole chunk included; a step of {w.n_stages * w.n_layers} such calls would take "
                    f"{w.n_stages * w.n_layers}x as long (extrapolated, not timed)"),
            tiny_stream_in_full=oracle_tiny_stream())
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling only: run a reduced number of layers (smaller arena for ncu captures)")
    ap.add_argument("--skip-cpu", action="store_true", help="profiling only: skip the CPU-oracle leg")
    ap.add_argument("--workload", default=WORKLOAD, choices=[n for n in W.CONFIG_ORDER if n != "tiny"],
                    help="extra: measure another of the benchmark's configurations (steady-state chunks)")
    ap.add_argument("--stream", action="store_true",
                    help="extra: also run the workload's whole stream once from empty banks and report its wall time")
    ap.add_argument("--skip-extra", action="store_true", help="skip the extra measurement at the paper's budget")
    ap.add_argument("--mode", default="replicas", choices=["replicas", "wavefront", "adjacent"],
                    help="replicas (default, the headline): every rank runs the whole path on its own GPU; wavefront: "
                         "the paper's stage-per-GPU pipeline over --gpus ranks (1, 2 or 4 for four stages); adjacent: "
                         "only the extra timings of the publish pass with and without q/k normalisation and of the "
                         "Euler update (one GPU; the small case the publish kernels are profiled on)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.mode == "wavefront":
        run_wavefront_mode(args)
    elif args.mode == "adjacent":
        import paper_2609_32540_b200 as P
        torch.cuda.set_device(0)
        print(json.dumps(dict(mode="adjacent", adjacent_steps=measure_adjacent_steps(
            P, torch.device("cuda:0"), 0, read_peaks()["hbm_gbs"]))), flush=True)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
