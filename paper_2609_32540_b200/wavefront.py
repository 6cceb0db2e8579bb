"""Renderer wavefront with one rank per denoising stage (Alg. 1, Phase B): plumbing only.

Round n: rank r (stage k = S - r) works on chunk i = n - r if that chunk exists.  It obtains the chunk's latent
(rank 0 draws noise, rank r > 0 receives what rank r - 1 sent in round n - 1), runs the chunk through its stage -
every layer's chunk attention against its OWN bank, which never leaves the rank, then the Euler update - and
hands the latent on (the last rank delivers the clean chunk).  The only traffic is one latent per chunk and hop,
sent point to point with torch.distributed (NCCL on GPUs, gloo in the CPU tests); no collective is involved.

Everything that computes is supplied by the caller (on a GPU: calls into the library through a Cache that was
created with n_stages = 1); this module holds the round arithmetic, the message order and the failure handling.
A rank that dies is noticed by its neighbours as an exception from the pending send or receive once the process
group's timeout expires; nothing here waits without a limit.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Optional

import torch
import torch.distributed as dist


def round_nodes(n: int, n_stages: int, n_chunks: int) -> list[tuple[int, int, int]]:
    """The active nodes of round n as (rank r, chunk i = n - r, stage k = S - r), 0 <= i < N_R."""
    return [(r, n - r, n_stages - r) for r in range(n_stages) if 0 <= n - r < n_chunks]


def n_rounds(n_stages: int, n_chunks: int) -> int:
    """N_R + S - 1 rounds empty the wavefront."""
    return n_chunks + n_stages - 1 if n_chunks > 0 else 0


@dataclass
class WavefrontStats:
    rounds: int = 0
    chunks: int = 0
    sent: int = 0
    received: int = 0


class StageRank:
    """One rank of the wavefront.

    obtain(i)      -> latent of chunk i at the highest noise level (rank 0 only: the noise sample)
    run_node(i, x) -> latent of chunk i after this rank's stage (attention layers + Euler update)
    deliver(i, x)  -> called on the last rank with the clean chunk
    Latents are tensors of one fixed shape and dtype (`like`), on the device the process group moves (CUDA
    tensors with NCCL, CPU tensors with gloo).
    """

    def __init__(self, rank: int, n_stages: int, n_chunks: int, like: torch.Tensor, *,
                 obtain: Optional[Callable[[int], torch.Tensor]], run_node: Callable[[int, torch.Tensor], torch.Tensor],
                 deliver: Optional[Callable[[int, torch.Tensor], None]] = None, group=None, first_chunk: int = 0):
        if not 0 <= rank < n_stages:
            raise ValueError("rank outside the stage range")
        if rank == 0 and obtain is None:
            raise ValueError("rank 0 needs a noise source")
        self.rank, self.n_stages, self.n_chunks = rank, n_stages, n_chunks
        self.stage = n_stages - rank          # k in the paper's numbering (S .. 1)
        self.like, self.group = like, group
        self.obtain, self.run_node, self.deliver = obtain, run_node, deliver
        self.first_chunk = first_chunk        # chunks first_chunk .. first_chunk + n_chunks - 1 (banks may be warm)
        self.stats = WavefrontStats()

    def run(self) -> WavefrontStats:
        pending = None                        # the send of the previous round, still in flight
        for n in range(n_rounds(self.n_stages, self.n_chunks)):
            i = n - self.rank
            if not 0 <= i < self.n_chunks:
                continue
            i += self.first_chunk
            if self.rank == 0:
                x = self.obtain(i)
            else:
                x = torch.empty_like(self.like)
                dist.recv(x, src=self.rank - 1, group=self.group, tag=i)
                self.stats.received += 1
            y = self.run_node(i, x)
            if pending is not None:
                pending.wait()                # the buffer of the previous send may be reused from here on
                pending = None
            if self.rank + 1 < self.n_stages:
                pending = dist.isend(y, dst=self.rank + 1, group=self.group, tag=i)
                self.stats.sent += 1
            elif self.deliver is not None:
                self.deliver(i, y)
            self.stats.rounds += 1
            self.stats.chunks += 1
        if pending is not None:
            pending.wait()
        return self.stats


class RendererStages:
    """What one rank of the stage-per-GPU renderer does with a chunk (Alg. 1 Phase B, "Read / Evaluate / Step /
    Write in place" on the rank that owns stage k): for each denoising stage the rank owns - one when there are as
    many ranks as stages, all S on a single rank, which is then the chunk-major order - every layer's chunk
    attention against the rank's own bank, Tail_H, and the Euler update of the chunk's latent.

    cache: a Cache created with n_stages = the number of stages this rank owns (bank index n_local-1 is the
    noisiest of them).  levels: per owned stage, in the order they run, (sigma_k, sigma_{k-1}).  io: ff_layer_io
    array of n_layers entries (device pointers of the layer inputs; the projections that would produce them are
    outside this library).  velocity: tensor shaped like the latent standing in for the forward's prediction.
    With a bookkeeping-only cache (no device) the calls are validated and counted and the update runs on the
    latent's own device with torch: the plumbing can be exercised on CPU ranks."""

    def __init__(self, cache, binding, levels, io, velocity: torch.Tensor, stream: int = 0, dry: bool = False):
        self.cache, self.B, self.levels, self.io = cache, binding, list(levels), io
        self.velocity, self.stream, self.dry = velocity, stream, dry
        self.layer_calls = 0

    def run_node(self, chunk: int, n_frames: int, first_frame_pos: int, anchor_slots, x: torch.Tensor) -> torch.Tensor:
        B = self.B
        n_local = len(self.levels)
        for j, (sigma_k, sigma_km1) in enumerate(self.levels):
            st = self.cache.ff_sched_run_node(n_local - 1 - j, chunk, n_frames, first_frame_pos, list(anchor_slots),
                                              self.io, self.stream)
            if st != B.FF_OK:
                raise B.FFError(st, f"ff_sched_run_node(chunk {chunk}, local stage {n_local - 1 - j})")
            self.layer_calls += self.cache.cfg.n_layers
            if self.dry:
                x = x - (sigma_k - sigma_km1) * self.velocity.to(x.dtype)
            else:
                code = {torch.float32: B.FF_F32, torch.bfloat16: B.FF_BF16}
                st = B.ff_euler_step(x.data_ptr(), self.velocity.data_ptr(), sigma_k, sigma_km1, x.numel(),
                                     code[x.dtype], code[self.velocity.dtype], x.data_ptr(), self.stream)
                if st != B.FF_OK:
                    raise B.FFError(st, "ff_euler_step")
        return x


@dataclass
class PlanStep:
    """One step of a clip's schedule: publish the clean KV of anchor `anchor` (its position on the timeline is
    `frame_pos`) into `slot`, or run renderer chunk `chunk` reading the anchors in `anchor_slots`."""
    kind: str                    # "anchor" | "chunk"
    anchor: int = -1
    slot: int = -1
    frame_pos: int = -1
    chunk: int = -1
    n_frames: int = 0
    first_frame_pos: int = 0
    anchor_slots: tuple = ()


def clip_plan(n_latents: int, chunk_frames: int, delta: int, n_anchor_slots: int, lookahead_chunks: int = 0):
    """The order of anchor publishes and renderer chunks for one clip (Alg. 1: Phase A feeds Phase B): chunk i reads
    the window Gamma(i) of three consecutive anchors (index sets from the library's host helpers); an anchor is
    published just before the first chunk that reads it, into slot `anchor mod n_anchor_slots`.

    lookahead_chunks = how many chunks beyond chunk i may still be in flight when chunk i enters (S - 1 for a
    wavefront over S stages, 0 for chunk-major order); the function checks that no publish overwrites a slot that
    one of those chunks still reads and raises ValueError otherwise (five slots are enough for the paper's budget).
    """
    from . import binding as B
    n_chunks = -(-n_latents // chunk_frames)
    windows = [B.ff_plan_window(i, n_latents, chunk_frames, delta) for i in range(n_chunks)]
    steps, published = [], {}
    for i in range(n_chunks):
        for m in windows[i]:
            if m in published:
                continue
            slot = m % n_anchor_slots
            for j in range(max(0, i - lookahead_chunks), i + 1):   # chunks in flight when this publish is enqueued
                for other in windows[j]:
                    if other != m and other % n_anchor_slots == slot and (other in published or j == i):
                        raise ValueError(f"anchor {m} would overwrite anchor {other}, still read by chunk {j}: "
                                         f"{n_anchor_slots} anchor slots are too few")
            published[m] = slot
            steps.append(PlanStep("anchor", anchor=m, slot=slot, frame_pos=B.ff_plan_anchor_position(n_latents, delta, m)))
        steps.append(PlanStep("chunk", chunk=i, n_frames=min(chunk_frames, n_latents - i * chunk_frames),
                              first_frame_pos=i * chunk_frames, anchor_slots=tuple(m % n_anchor_slots for m in windows[i])))
    return steps
