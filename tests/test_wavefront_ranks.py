"""Stage-per-rank wavefront (Alg. 1 Phase B) on CPU ranks with gloo: round arithmetic, message order, the cache's
call-order rules on every rank (bookkeeping-only caches), and a rank that dies between steps."""
import os
import socket
import sys
from datetime import timedelta

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import paper_defs as PD  # noqa: E402


def test_round_nodes_match_the_papers_wavefront():
    from paper_2609_32540_b200 import wavefront as Wf
    S, N = 4, 27
    ref = PD.wavefront_rounds(N, S)          # the oracle's statement of Phase B: per round the (chunk, stage) pairs
    assert Wf.n_rounds(S, N) == len(ref) == 30
    seen = {}
    for n in range(Wf.n_rounds(S, N)):
        nodes = Wf.round_nodes(n, S, N)
        assert sorted((i, k) for _, i, k in nodes) == sorted(ref[n])
        assert len({r for r, _, _ in nodes}) == len(nodes) <= S
        for r, i, k in nodes:
            assert i == n - r and k == S - r and 0 <= i < N
            # dependencies of node (i, k): (i, k+1) ran one round earlier on rank r-1, (i-1, k) one round earlier here
            if r > 0:
                assert seen[(i, k + 1)] == n - 1
            if i > 0:
                assert seen[(i - 1, k)] == n - 1
            seen[(i, k)] = n
    assert len(seen) == S * N
    assert Wf.round_nodes(0, S, N) == [(0, 0, 4)] and Wf.round_nodes(29, S, N) == [(3, 26, 1)]
    assert Wf.n_rounds(4, 0) == 0


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n_chunks, die_at, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world, timeout=timedelta(seconds=8))
    import ff_workloads as W
    import paper_2609_32540_b200 as P
    from paper_2609_32540_b200 import binding as B
    from paper_2609_32540_b200 import wavefront as Wf
    w = W.scaled(W.CONFIGS["tiny"], anchor_policy="none", n_anchor_slots=0, n_layers=2)
    # every rank owns ONE stage: its bank never leaves the rank
    cache = B.Cache(B.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h,
                                  grid_w=w.grid_w, chunk_frames=w.chunk_frames, n_stages=1,
                                  history_chunks=w.history_chunks, n_anchor_slots=0, max_visible_anchors=0,
                                  device=B.FF_DEVICE_NONE), None, 0)
    sig = PD.sigma_schedule(world, 5.0)
    k = world - rank
    like = torch.zeros(8, dtype=torch.float64)
    log = []

    def run_node(i, x):
        if die_at is not None and rank == die_at[0] and i == die_at[1]:
            raise RuntimeError("injected failure between steps")
        io = B.make_io([(16, 16, 16, 16)] * w.n_layers)
        st = cache.ff_sched_run_node(0, i, 1, i, [], io)     # all layers against the local bank, then Tail_H
        assert st == B.FF_OK, st
        log.append(i)
        # stand-in for the Euler update with a velocity that depends on chunk and stage
        return x - (sig[k] - sig[k - 1]) * float(10 * i + k)

    delivered = {}
    sr = Wf.StageRank(rank, world, n_chunks, like, obtain=(lambda i: torch.full_like(like, float(i))) if rank == 0 else None,
                      run_node=run_node, deliver=lambda i, x: delivered.__setitem__(i, x.clone()))
    try:
        stats = sr.run()
        ring = cache.ff_cache_ring_state(0, 0)
        q.put((rank, "ok", stats.chunks, stats.sent, stats.received, log, {i: float(x[0]) for i, x in delivered.items()},
               ring["next_chunk"]))
    except Exception as e:  # noqa: BLE001
        q.put((rank, "error", type(e).__name__, str(e)[:80]))
    finally:
        try:
            dist.destroy_process_group()
        except Exception:  # noqa: BLE001
            pass


def _spawn(world, n_chunks, die_at=None):
    from paper_2609_32540_b200 import build
    build.build()          # the ranks load the shared library; nvcc cross-compiles without a GPU
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, n_chunks, die_at, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    return res


@pytest.mark.parametrize("world", [2, 3])
def test_chunks_pass_through_every_stage_in_order(world):
    n_chunks = 5
    res = _spawn(world, n_chunks)
    sig = PD.sigma_schedule(world, 5.0)
    for rank, status, *rest in res:
        assert status == "ok", rest
        chunks, sent, received, log, delivered, next_chunk = rest
        assert chunks == n_chunks and log == list(range(n_chunks)) and next_chunk == n_chunks
        assert sent == (n_chunks if rank < world - 1 else 0) and received == (n_chunks if rank > 0 else 0)
        if rank == world - 1:
            for i in range(n_chunks):
                want = float(i) - sum((sig[k] - sig[k - 1]) * (10 * i + k) for k in range(world, 0, -1))
                assert abs(delivered[i] - want) < 1e-12
        else:
            assert delivered == {}


def test_a_rank_that_dies_between_steps_ends_the_others_with_an_error():
    res = _spawn(2, 6, die_at=(1, 2))
    by_rank = {r[0]: r for r in res}
    assert by_rank[1][1] == "error" and by_rank[1][2] == "RuntimeError"
    # rank 0 learns of it from its pending send or the next one: an exception, not a hang
    assert by_rank[0][1] == "error"


def _bench_rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world, timeout=timedelta(seconds=20))
    try:
        import bench
        import ff_workloads as W
        import paper_2609_32540_b200 as P
        w = W.scaled(W.CONFIGS["tiny"], n_stages=4, n_layers=3)
        res = bench.pipeline_run(P, w, world, rank, steps=5, warmup=4, device_index=None)
        q.put((rank, "ok", res))
    except Exception as e:  # noqa: BLE001
        q.put((rank, "error", f"{type(e).__name__}: {e}"[:200]))
    finally:
        try:
            dist.destroy_process_group()
        except Exception:  # noqa: BLE001
            pass


@pytest.mark.parametrize("world", [1, 2])
def test_bench_wavefront_mode_runs_the_same_code_on_cpu_ranks(world):
    """bench.py --mode wavefront, as launched on GPUs, is pipeline_run on every rank; here the same function runs on
    gloo ranks over bookkeeping-only caches: four denoising stages shared by the ranks, every rank's call sequence
    accepted by its own cache, the latents handed on in order, the clean chunks delivered by the last rank."""
    from paper_2609_32540_b200 import build
    build.build()
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_bench_rank_main, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    for rank, status, r in res:
        assert status == "ok", r
        n_local = 4 // world
        assert r["stages_per_rank"] == n_local and r["chunks"] == 5
        assert r["layer_calls"] == 5 * n_local * 3 and r["advances"] == 5 * n_local
        assert r["sent"] == (5 if rank < world - 1 else 0) and r["received"] == (5 if rank > 0 else 0)
        assert r["delivered"] == (list(range(9)) if rank == world - 1 else [])   # warm-up chunks included
        assert r["flops"] > 0 and r["ms"] > 0


def test_clip_plan_follows_the_papers_windows_and_guards_slot_reuse():
    from paper_2609_32540_b200 import build, wavefront as Wf
    build.build()
    import ff_workloads as W
    L, B_R, delta = 81, 3, 10
    steps = Wf.clip_plan(L, B_R, delta, n_anchor_slots=5, lookahead_chunks=3)
    chunks = [s for s in steps if s.kind == "chunk"]
    anchors = [s for s in steps if s.kind == "anchor"]
    assert len(chunks) == 27 and [a.anchor for a in anchors] == list(range(9))
    assert [a.frame_pos for a in anchors] == PD.anchor_positions(L, delta)
    slot_pos = {}
    for s in steps:
        if s.kind == "anchor":
            slot_pos[s.slot] = s.frame_pos
        else:
            # what the chunk reads, as timeline positions, is the paper's Gamma(i) (oracle statement)
            assert sorted(slot_pos[x] for x in s.anchor_slots) == sorted(PD.gamma_paper(s.chunk, L, B_R, delta))
    # the same recipe the synthetic workloads use
    w = W.PAPER_480P
    assert [tuple(W.anchor_slot(w, m) for m in W.visible_anchor_ids(w, c.chunk)) for c in chunks] == [c.anchor_slots for c in chunks]
    # chunk-major order: a window's three slots are enough, the next window replaces anchors no chunk reads any more
    assert len(Wf.clip_plan(L, B_R, delta, n_anchor_slots=3)) == 27 + 9
    assert len(Wf.clip_plan(21, 3, 10, n_anchor_slots=3)) == 7 + 3
    with pytest.raises(ValueError):
        Wf.clip_plan(L, B_R, delta, n_anchor_slots=2)                       # a window does not fit
    # a four-stage wavefront keeps chunks of two windows in flight: five distinct anchors
    for slots in (3, 4):
        with pytest.raises(ValueError):
            Wf.clip_plan(L, B_R, delta, n_anchor_slots=slots, lookahead_chunks=3)
