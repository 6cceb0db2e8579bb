"""Behaviour of the C ABI on a GPU: execution orders, isolation, host-buffer and scheduler entry points, error
reporting, and the bounded-wait path."""
import numpy as np
import pytest
import torch

import ff_workloads as W
from oracle import ff_oracle as O
from oracle import paper_defs as PD
from tests import ff_harness as Hn

pytestmark = pytest.mark.gpu

MID = W.Workload("mid", 2, 3, 128, 9, 11, 2, 4, 2, 12, 1, 4, "every", 4)   # 4 stages, 6 chunks of 198 tokens


def _inputs(w, seed, chunk, stage, layer, n_frames):
    return tuple(t.cuda() for t in W.qkv(w, seed, chunk, stage, layer, n_frames))


def _run(w, order, poison_between=False, impl=1):
    """Runs the whole stream in chunk-major or wavefront order; returns outputs and the final arena bytes."""
    gpu = Hn.GpuCache(w, O.BF16, impl)
    outs = {}
    events = {e.chunk: e for e in W.trace(w) if e.kind == "chunk"}
    anchors = [e for e in W.trace(w) if e.kind == "anchor"]
    for a in anchors:   # all anchors first: slots are sized so that none is recycled (planner finished, Phase A)
        for l in range(w.n_layers):
            k, v = W.anchor_kv(w, 0, a.anchor_id, l)
            assert gpu.anchor_publish(a.slot, a.frame_pos, l, k.cuda(), v.cuda()) == 0
    if order == "chunk":
        nodes = [(i, k) for i in range(w.n_chunks) for k in range(w.n_stages, 0, -1)]
    else:
        nodes = [n for rnd in PD.wavefront_rounds(w.n_chunks, w.n_stages) for n in rnd]
    for (i, k) in nodes:
        ev, stage = events[i], k - 1
        io, keep = [], []
        for l in range(w.n_layers):
            q, kk, v = _inputs(w, 0, i, stage, l, ev.n_frames)
            out = torch.full_like(q, float("nan"))
            keep.append((q, kk, v, out))
            io.append((q.data_ptr(), kk.data_ptr(), v.data_ptr(), out.data_ptr()))
            outs[(i, stage, l)] = out
        if poison_between:
            # everything this node must not read: the other stages' rings and the slot it is about to overwrite
            H = w.history_chunks
            for s2 in range(w.n_stages):
                for l in range(w.n_layers):
                    for sl in range(H + 1):
                        if s2 != stage or sl == i % (H + 1):
                            _poison_slot(gpu, s2, l, sl, save=(s2 != stage))
        st = gpu.cache.ff_sched_run_node(stage, i, ev.n_frames, ev.first_frame_pos, ev.anchor_slots, io, gpu.stream)
        assert st == 0, st
        torch.cuda.synchronize()
        if poison_between:
            _restore_slots(gpu)
    st, word = gpu.cache.ff_cache_status(gpu.stream)
    assert st == 0 and word == 0
    return outs, gpu


_saved = []


def _slot_views(gpu, stage, layer, slot):
    info = gpu.cache.ff_cache_slot_ptr(0, stage, layer, slot)
    views = []
    for ptr in (info["k"], info["v"]):
        off = ptr - gpu.arena.data_ptr()
        flat = gpu.arena[off:].view(torch.bfloat16)
        st = info["strides"]
        views.append(torch.as_strided(flat, (info["capacity_tokens"], gpu.w.n_heads, gpu.w.head_dim), st))
    return views


def _poison_slot(gpu, stage, layer, slot, save):
    for v in _slot_views(gpu, stage, layer, slot):
        if save:
            _saved.append((v, v.clone()))
        v.fill_(float("nan"))


def _restore_slots(gpu):
    while _saved:
        v, data = _saved.pop()
        v.copy_(data)


def test_wavefront_order_is_bit_identical_to_chunk_major():
    """Alg. 1 Phase B order (node (i,k) in round i + S - k) against chunk-major order: per-stage rings make the
    outputs and every ring slot identical bit for bit."""
    a, ga = _run(MID, "chunk")
    b, gb = _run(MID, "wave")
    assert a.keys() == b.keys() and len(a) == MID.n_chunks * MID.n_stages * MID.n_layers
    for key in a:
        assert torch.equal(a[key], b[key]), key
    for stage in range(MID.n_stages):
        assert ga.cache.ff_cache_ring_state(stage, 0) == gb.cache.ff_cache_ring_state(stage, 0)
        for l in range(MID.n_layers):
            for sl in range(MID.history_chunks + 1):
                for x, y in zip(_slot_views(ga, stage, l, sl), _slot_views(gb, stage, l, sl)):
                    n = ga.cache.ff_cache_ring_state(stage, l)["slot_tokens"][sl]
                    assert torch.equal(x[:n], y[:n])
    ga.close(); gb.close()


def test_other_stages_and_evicted_slot_are_never_read():
    """NaN in every other stage's ring and in the slot about to be overwritten changes no output bit."""
    a, ga = _run(MID, "chunk")
    b, gb = _run(MID, "chunk", poison_between=True)
    for key in a:
        assert torch.isfinite(b[key].float()).all(), key
        assert torch.equal(a[key], b[key]), key
    ga.close(); gb.close()


def test_tensor_core_kernel_agrees_with_cuda_core_kernel():
    a, ga = _run(MID, "chunk", impl=1)
    b, gb = _run(MID, "chunk", impl=2)
    worst = max((a[k].float() - b[k].float()).abs().max().item() for k in a)
    assert worst <= 1e-2, worst
    ga.close(); gb.close()


def test_host_buffer_and_scheduler_entry_points_match_device_entry_point():
    w = W.Workload("hostv", 2, 2, 64, 8, 8, 1, 2, 2, 4, 1, 2, "ahead", 3, clip_anchor_pos=False)
    res = {}
    for mode in ("device", "host", "sched", "sched_host"):
        gpu = Hn.GpuCache(w, O.BF16, 1)
        outs = {}
        for ev in W.trace(w):
            if ev.kind == "anchor":
                for l in range(w.n_layers):
                    k, v = W.anchor_kv(w, 0, ev.anchor_id, l)
                    assert gpu.anchor_publish(ev.slot, ev.frame_pos, l, k.cuda(), v.cuda()) == 0
                continue
            cpu = {(s, l): W.qkv(w, 0, ev.chunk, s, l, ev.n_frames) for s in range(w.n_stages) for l in range(w.n_layers)}
            if mode in ("device", "sched"):
                dev = {key: tuple(t.cuda() for t in val) + (torch.full_like(val[0], float("nan")).cuda(),)
                       for key, val in cpu.items()}
            else:
                dev = {key: tuple(t.pin_memory() for t in val) + (torch.full_like(val[0], float("nan")).pin_memory(),)
                       for key, val in cpu.items()}
            ptrs = {key: tuple(t.data_ptr() for t in val) for key, val in dev.items()}
            if mode in ("sched", "sched_host"):
                io = [ptrs[(s, l)] for s in range(w.n_stages) for l in range(w.n_layers)]
                fn = gpu.cache.ff_sched_run_chunk if mode == "sched" else gpu.cache.ff_sched_run_chunk_host
                assert fn(ev.chunk, ev.n_frames, ev.first_frame_pos, ev.anchor_slots, io, gpu.stream) == 0
            else:
                fn = gpu.cache.ff_chunk_forward_attn if mode == "device" else gpu.cache.ff_chunk_forward_attn_host
                for s in reversed(range(w.n_stages)):
                    for l in range(w.n_layers):
                        q, k, v, o = ptrs[(s, l)]
                        assert fn(s, l, ev.chunk, ev.n_frames, ev.first_frame_pos, q, k, v, ev.anchor_slots, o,
                                  gpu.stream) == 0
                    assert gpu.cache.ff_cache_advance(s) == 0
            torch.cuda.synchronize()
            for key, val in dev.items():
                outs[(ev.chunk,) + key] = val[3].cpu().clone()
        res[mode] = outs
        gpu.close()
    for mode in ("host", "sched", "sched_host"):
        for key in res["device"]:
            assert torch.equal(res["device"][key], res[mode][key]), (mode, key)


def test_error_codes_enqueue_nothing_and_leave_state_unchanged():
    from paper_2609_32540_b200 import binding as B
    w = W.CONFIGS["tiny"]
    gpu = Hn.GpuCache(w, O.BF16, 1)
    q, k, v = _inputs(w, 0, 0, 0, 0, 1)
    out = torch.empty_like(q)
    c = gpu.cache
    args = (q.data_ptr(), k.data_ptr(), v.data_ptr())
    before = c.ff_cache_counters()
    assert c.ff_chunk_forward_attn(0, 0, 1, 1, 1, *args, [], out.data_ptr(), gpu.stream) == B.FF_ERR_STATE     # chunk 1 before 0
    assert c.ff_chunk_forward_attn(0, 0, 0, 1, 0, *args, [0], out.data_ptr(), gpu.stream) == B.FF_ERR_STATE    # anchor not published
    assert c.ff_chunk_forward_attn(0, 0, 0, 2, 0, *args, [], out.data_ptr(), gpu.stream) == B.FF_ERR_INVALID_ARG  # > B_R frames
    assert c.ff_chunk_forward_attn(5, 0, 0, 1, 0, *args, [], out.data_ptr(), gpu.stream) == B.FF_ERR_INVALID_ARG
    assert c.ff_chunk_forward_attn(0, 0, 0, 1, 0, args[0] + 2, args[1], args[2], [], out.data_ptr(),
                                   gpu.stream) == B.FF_ERR_INVALID_ARG                                        # misaligned
    assert c.ff_chunk_forward_attn(0, 0, 0, 1, 0, *args, [0, 1], out.data_ptr(), gpu.stream) == B.FF_ERR_INVALID_ARG
    assert c.ff_cache_advance(0) == B.FF_ERR_STATE                                                           # nothing appended
    assert c.ff_anchor_publish(9, 0, 0, k.data_ptr(), v.data_ptr(), gpu.stream) == B.FF_ERR_INVALID_ARG
    assert c.ff_cache_counters() == before
    assert c.ff_cache_ring_state(0)["next_chunk"] == 0
    # the same layer twice for one chunk is refused
    assert c.ff_chunk_forward_attn(0, 0, 0, 1, 0, *args, [], out.data_ptr(), gpu.stream) == B.FF_OK
    assert c.ff_chunk_forward_attn(0, 0, 0, 1, 0, *args, [], out.data_ptr(), gpu.stream) == B.FF_ERR_STATE
    # arena too small / misaligned
    cfg = gpu.cfg
    with pytest.raises(B.FFError) as e:
        B.Cache(cfg, gpu.arena.data_ptr(), gpu.nbytes - 1)
    assert e.value.status == B.FF_ERR_OOM
    with pytest.raises(B.FFError) as e:
        B.Cache(cfg, gpu.arena.data_ptr() + 8, gpu.nbytes)
    assert e.value.status == B.FF_ERR_INVALID_ARG
    # reset empties the banks
    assert c.ff_cache_reset() == 0 and c.ff_cache_ring_state(0)["slot_chunk"] == [-1, -1, -1]
    gpu.close()


def test_expired_device_wait_is_reported_and_the_context_stays_usable():
    """A wait that nothing will ever satisfy runs into its (1 ms) limit: the kernel returns, the status word says
    so, and the next layer-call on the same cache is still correct."""
    from paper_2609_32540_b200 import binding as B
    w = W.CONFIGS["tiny"]
    gpu = Hn.GpuCache(w, O.BF16, 1)
    assert gpu.cache.ff_debug_wait_probe(1_000_000, gpu.stream) == 0
    st, word = gpu.cache.ff_cache_status(gpu.stream)
    assert st == B.FF_ERR_TIMEOUT and word == 0x1FF
    st, word = gpu.cache.ff_cache_status(gpu.stream)
    assert st == 0 and word == 0                      # reading clears it
    orc = Hn.make_oracle(W.scaled(w, anchor_policy="none"), O.BF16)
    q, k, v = W.qkv(w, 0, 0, 0, 0, 1)
    st, out = gpu.forward(0, 0, 0, 1, 0, q.cuda(), k.cuda(), v.cuda(), [])
    assert st == 0
    so, want = orc.chunk_forward(0, 0, 0, 1, 0, q.float().numpy(), k.float().numpy(), v.float().numpy())
    torch.cuda.synchronize()
    Hn.compare_outputs(out, want, O.BF16, "after an expired wait")
    gpu.close()


def test_auto_kernel_choice_follows_the_query_tile_count():
    """FF_ATTN_AUTO with head_dim 128: the kernel on CTA pairs when four-tile units waste at most 4 % more query-tile
    slots than two-tile units (8 tiles per head: none; 5 tiles: 8 slots against 6), the one-CTA kernel otherwise;
    forcing a kernel is honoured; head_dim 64 has only the one-CTA kernel."""
    from paper_2609_32540_b200 import binding as B
    cases = [(8 * 128, 0, "cta_pair"), (5 * 128, 0, "one_cta"), (8 * 128, 1, "one_cta"), (5 * 128, 3, "cta_pair")]
    for n_tok, impl, want in cases:
        w = W.Workload("choice", 1, 2, 128, 8, n_tok // 8, 1, 1, 0, 1, 0, 0, "none", 1)
        gpu = Hn.GpuCache(w, O.BF16, attn_impl=impl)
        q, k, v = (t.cuda() for t in W.qkv(w, 0, 0, 0, 0, 1))
        st, out = gpu.forward(0, 0, 0, 1, 0, q, k, v, [])
        assert st == 0
        torch.cuda.synchronize()
        c = gpu.cache.ff_cache_kernel_choice()
        assert c[want] == 1 and c["one_cta" if want == "cta_pair" else "cta_pair"] == 0, (n_tok, impl, c)
        orc = Hn.make_oracle(w, O.BF16)
        so, truth = orc.chunk_forward(0, 0, 0, 1, 0, q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy(), [])
        Hn.compare_outputs(out, truth, O.BF16, f"kernel choice {n_tok} {impl}")
        gpu.close()
    w64 = W.scaled(W.CONFIGS["tiny"], anchor_policy="none", n_anchor_slots=0)
    with pytest.raises(B.FFError) as e:
        Hn.GpuCache(w64, O.BF16, attn_impl=3)
    assert e.value.status == B.FF_ERR_UNSUPPORTED


def test_profile_hooks_time_both_kernels():
    w = W.CONFIGS["tiny"]
    gpu = Hn.GpuCache(w, O.BF16, 1)
    assert gpu.cache.ff_cache_profile_begin(4) == 0
    q, k, v = _inputs(w, 0, 0, 0, 0, 1)
    st, out = gpu.forward(0, 0, 0, 1, 0, q, k, v, [])
    assert st == 0
    p = gpu.cache.ff_cache_profile_end(gpu.stream)
    assert p["attn_launches"] == 1 and p["attn_ms"] > 0 and p["publish_ms"] > 0
    gpu.close()


def test_non_default_stream_and_two_caches_interleaved():
    """Two independent caches driven call by call, alternately, on one side stream (the kernels are launched as
    programmatic dependents: each must still be ordered after whatever precedes it on that stream, here a
    kernel of the OTHER cache); both must match their oracles, cache contents bit for bit."""
    side = torch.cuda.Stream()
    wa = W.scaled(W.CONFIGS["tiny"], anchor_policy="none", n_anchor_slots=0, n_layers=2)
    wb = W.Workload("other", 1, 3, 128, 5, 9, 2, 2, 1, 8, 0, 0, "none", 4)
    with torch.cuda.stream(side):
        caches = [(wa, Hn.GpuCache(wa, O.BF16, attn_impl=1), Hn.make_oracle(wa, O.BF16), 21),
                  (wb, Hn.GpuCache(wb, O.BF16, attn_impl=1), Hn.make_oracle(wb, O.BF16), 22)]
        assert all(g.stream == side.cuda_stream for _, g, _, _ in caches)
        n_chunks = min(wa.n_chunks, wb.n_chunks)
        for i in range(n_chunks):
            for stage in reversed(range(2)):
                pending = []
                for l in range(2):
                    for w, gpu, orc, seed in caches:
                        if l >= w.n_layers:
                            continue
                        nf = w.chunk_frames_of(i)
                        q, k, v = W.qkv(w, seed, i, stage, l, nf)
                        st, out = gpu.forward(stage, l, i, nf, i * w.chunk_frames, q.cuda(), k.cuda(), v.cuda(), [])
                        assert st == 0
                        pending.append((w, gpu, orc, l, nf, q, k, v, out))
                side.synchronize()
                for w, gpu, orc, l, nf, q, k, v, out in pending:
                    so, want = orc.chunk_forward(stage, l, i, nf, i * w.chunk_frames, q.float().numpy(), k.float().numpy(),
                                                 v.float().numpy())
                    assert so == 0
                    Hn.compare_outputs(out, want, O.BF16, f"{w.name} chunk {i} stage {stage} layer {l}")
                    Hn._compare_slot_mapped(gpu, orc, 0, stage, l, l, i % (w.history_chunks + 1))
                for w, gpu, orc, _ in caches:
                    assert gpu.cache.ff_cache_advance(stage) == 0 and orc.advance(stage) == 0
        for _, gpu, _, _ in caches:
            st, word = gpu.cache.ff_cache_status(gpu.stream)
            assert st == 0 and word == 0
            gpu.close()


def test_torch_convenience_layer_matches_the_oracle_and_rejects_bad_tensors():
    from paper_2609_32540_b200 import torch_api as T
    from paper_2609_32540_b200 import binding as B
    w = W.scaled(W.CONFIGS["tiny"], anchor_policy="ahead")
    c = T.ChunkAttentionCache(0, n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h,
                              grid_w=w.grid_w, chunk_frames=w.chunk_frames, n_stages=w.n_stages,
                              history_chunks=w.history_chunks, n_anchor_slots=w.n_anchor_slots, max_visible_anchors=1)
    orc = Hn.make_oracle(w, O.BF16)
    for ev in W.trace(w, 3):
        if ev.kind == "anchor":
            k, v = W.anchor_kv(w, 5, ev.anchor_id, 0)
            c.publish_anchor(ev.slot, ev.frame_pos, 0, k.cuda(), v.cuda())
            assert orc.anchor_publish(ev.slot, ev.frame_pos, 0, k.float().numpy(), v.float().numpy()) == 0
            continue
        for stage in reversed(range(w.n_stages)):
            q, k, v = W.qkv(w, 5, ev.chunk, stage, 0, ev.n_frames)
            out = c.forward(stage, 0, ev.chunk, ev.first_frame_pos, q.cuda(), k.cuda(), v.cuda(), ev.anchor_slots)
            so, want = orc.chunk_forward(stage, 0, ev.chunk, ev.n_frames, ev.first_frame_pos, q.float().numpy(),
                                         k.float().numpy(), v.float().numpy(), ev.anchor_slots)
            assert so == 0
            c.check_device_status()
            Hn.compare_outputs(out, want, O.BF16, f"chunk {ev.chunk} stage {stage}")
            c.advance(stage), orc.advance(stage)
    q, k, v = (t.cuda() for t in W.qkv(w, 5, 3, 1, 0, 1))
    with pytest.raises(ValueError):
        c.forward(1, 0, 3, 3, q.float(), k, v)                       # wrong dtype
    with pytest.raises(ValueError):
        c.forward(1, 0, 3, 3, q[:, :1], k, v)                        # wrong shape
    with pytest.raises(ValueError):
        c.forward(1, 0, 3, 3, q.cpu(), k, v)                         # wrong device
    with pytest.raises(B.FFError) as e:
        c.forward(1, 0, 7, 7, q, k, v)                               # not the stage's next chunk
    assert e.value.status == B.FF_ERR_STATE
    x = torch.randn(1001, device="cuda")
    vel = torch.randn(1001, device="cuda").bfloat16()
    y = T.euler_step(x, vel, 0.9375, 0.8333)
    want = O.euler_step(x.cpu().numpy(), vel.float().cpu().numpy(), np.float32(0.9375), np.float32(0.8333))
    assert np.array_equal(y.cpu().numpy(), want)
    c.close()
