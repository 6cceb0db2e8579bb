"""One wavefront round per launch group (Alg. 1 Phase B on one device): the nodes of a round share one attention
launch; results must equal the oracle's node-by-node run, cache bit for bit."""
import pytest
import torch

import ff_workloads as W
from oracle import ff_oracle as O
from tests import ff_harness as Hn

pytestmark = pytest.mark.gpu

TINY = W.CONFIGS["tiny"]


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2609_32540_b200 import binding
    binding.load()   # fails loudly when the extension is missing


@pytest.mark.parametrize("dtype,impl,round_call", [(O.BF16, 1, True), (O.BF16, 1, False), (O.BF16, 2, True),
                                                   (O.F32, 2, False)])
def test_tiny_wavefront_full_parity(dtype, impl, round_call):
    stats, gpu, orc = Hn.run_wavefront(TINY, dtype, attn_impl=impl, seed=0, use_round_call=round_call)
    assert len(stats) == TINY.n_chunks * TINY.n_stages * TINY.n_layers
    c = gpu.cache.ff_cache_counters()
    assert c["layer_calls"] == len(stats) and c["advances"] == TINY.n_chunks * TINY.n_stages
    gpu.close()


def test_four_stage_ragged_multi_tile_wavefront():
    """Four stages, d = 128, several heads, token counts off the tile grid, a short last chunk (so the nodes of a
    round differ in query rows AND in visible keys), two anchors per window: every CTA's work list crosses items."""
    w = W.Workload("wave_ragged", 2, 3, 128, 9, 23, 2, 4, 2, 11, 2, 3, "bracket", 4)
    stats, gpu, orc = Hn.run_wavefront(w, O.BF16, attn_impl=1, seed=6, rows_fn=lambda n: W.sample_rows(n, 24, 2))
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    c = gpu.cache.ff_cache_counters()
    # per layer and round: one publish per node plus the attention launch (+ at most one merge launch)
    rounds = w.n_chunks + w.n_stages - 1
    assert c["kernel_launches"] - c["anchor_publishes"] - c["layer_calls"] <= 2 * rounds * w.n_layers
    gpu.close()


def test_batch_call_rejects_bad_batches_and_changes_nothing():
    w = W.scaled(TINY, anchor_policy="none")
    gpu = Hn.GpuCache(w, O.BF16, attn_impl=1)
    q, k, v = (t.cuda() for t in W.qkv(w, 0, 0, 0, 0))
    out = torch.empty_like(q)
    item = dict(stage=1, chunk_index=0, n_frames=1, first_frame_pos=0, q=q.data_ptr(), k=k.data_ptr(), v=v.data_ptr(),
                out=out.data_ptr(), anchor_slots=[])
    before = gpu.cache.ff_cache_ring_state(1, 0)
    P = gpu.P
    assert gpu.cache.ff_batch_forward_attn(0, [item, dict(item)], gpu.stream) == P.FF_ERR_STATE   # same chunk twice
    bad = dict(item, stage=0, chunk_index=3)                                                         # not next chunk
    assert gpu.cache.ff_batch_forward_attn(0, [item, bad], gpu.stream) == P.FF_ERR_STATE
    assert gpu.cache.ff_batch_forward_attn(0, [], gpu.stream) == P.FF_ERR_INVALID_ARG
    assert gpu.cache.ff_batch_forward_attn(0, [dict(item, stage=s % 2) for s in range(3)], gpu.stream) != P.FF_OK
    assert gpu.cache.ff_cache_ring_state(1, 0) == before and gpu.cache.ff_cache_counters()["layer_calls"] == 0
    ok = dict(item, stage=0)
    assert gpu.cache.ff_batch_forward_attn(0, [item, ok], gpu.stream) == P.FF_OK
    torch.cuda.synchronize()
    assert gpu.cache.ff_cache_counters()["layer_calls"] == 2
    gpu.close()


def test_full_size_480p_wavefront_round_sampled():
    """The headline shape, four nodes per round at full token counts, two followed layers, sampled rows."""
    w = W.scaled(W.CONFIGS["wan1p3b_480p"], n_layers=3, total_frames=18)
    stats, gpu, orc = Hn.run_wavefront(w, O.BF16, attn_impl=1, seed=8, check_layers=[0, 2], pooled=True,
                                       rows_fn=lambda n: W.sample_rows(n, 4, 3), compare_cache=False)
    assert stats
    gpu.close()


@pytest.mark.parametrize("group,impl,dtype", [(3, 1, O.BF16), (6, 1, O.BF16), (4, 2, O.F32)])
def test_clip_at_once_under_the_chunkwise_causal_mask(group, impl, dtype):
    """Consecutive chunks of one stage in one launch (Sec. 3: the full clip at once with a chunk-wise causal mask):
    a later chunk of the group reads what the earlier ones publish in the same batch.  Tiny config in full."""
    w = W.scaled(TINY, n_anchor_slots=3)   # one slot per anchor: the planner's pass precedes the renderer's
    stats, gpu, orc = Hn.run_packed_clip(w, group, dtype, attn_impl=impl, seed=1)
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()


def test_clip_at_once_ragged_multi_tile():
    w = W.Workload("clip_ragged", 2, 3, 128, 9, 23, 2, 2, 2, 13, 2, 5, "bracket", 4)
    stats, gpu, orc = Hn.run_packed_clip(w, 4, O.BF16, attn_impl=1, seed=3, rows_fn=lambda n: W.sample_rows(n, 16, 4))
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()


def test_whole_clip_in_one_launch_tiny_and_ragged():
    """group = N_R: every chunk of a stage shares one attention launch per layer.  More layer-calls than travel as
    launch arguments, so the kernel reads its per-call descriptors from the table in the arena."""
    w = W.scaled(TINY, total_frames=11, n_anchor_slots=4)
    assert w.n_chunks == 11
    for impl, dtype in ((1, O.BF16), (2, O.F32)):
        stats, gpu, orc = Hn.run_packed_clip(w, w.n_chunks, dtype, attn_impl=impl, seed=2)
        assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
        c = gpu.cache.ff_cache_counters()
        if impl == 1:   # per (stage, layer): two publish launches (8 + 3 calls), one attention launch, at most one merge
            assert c["kernel_launches"] - c["anchor_publishes"] <= w.n_stages * w.n_layers * 4
        gpu.close()
    w = W.Workload("clip_ragged_whole", 2, 3, 128, 9, 23, 2, 2, 2, 19, 2, 6, "bracket", 4)   # 10 chunks, the last short
    assert w.n_chunks == 10 and w.chunk_frames_of(9) == 1
    stats, gpu, orc = Hn.run_packed_clip(w, w.n_chunks, O.BF16, attn_impl=1, seed=5, rows_fn=lambda n: W.sample_rows(n, 16, 4))
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()


def test_cta_pair_kernel_in_batched_launches():
    """The kernel on CTA pairs under the two batched forms: wavefront rounds (four nodes per launch, ragged shapes,
    a short last chunk) and a whole clip in one launch (descriptor table)."""
    w = W.Workload("pair_wavefront", 2, 3, 128, 9, 23, 2, 4, 2, 11, 2, 6, "bracket", 4)
    stats, gpu, orc = Hn.run_wavefront(w, O.BF16, attn_impl=3, seed=6, rows_fn=lambda n: W.sample_rows(n, 16, 6))
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()
    w = W.Workload("pair_clip", 2, 3, 128, 9, 23, 2, 2, 2, 19, 2, 6, "bracket", 4)
    stats, gpu, orc = Hn.run_packed_clip(w, w.n_chunks, O.BF16, attn_impl=3, seed=7, rows_fn=lambda n: W.sample_rows(n, 16, 7))
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()


def test_whole_81_latent_clip_in_one_launch_at_480p_token_counts():
    """The paper's worked example at full 480p token counts (27 chunks, H = 5, three anchors per window), one stage
    and two layers: ONE attention launch per layer over all 27 chunks; sampled rows of every chunk against the
    chunk-by-chunk oracle, every published slot bit for bit."""
    w = W.scaled(W.PAPER_480P, n_layers=2, n_stages=1, n_anchor_slots=9)
    assert w.n_chunks == 27
    stats, gpu, orc = Hn.run_packed_clip(w, 27, O.BF16, attn_impl=1, seed=9, rows_fn=lambda n: W.sample_rows(n, 3, 9))
    assert len(stats) == 27 * 2
    gpu.close()


def test_same_stage_batch_needs_enough_slots():
    w = W.scaled(TINY, anchor_policy="none")
    gpu = Hn.GpuCache(w, O.BF16, attn_impl=1, max_batch=4)          # default bank: H + 1 slots
    q, k, v = (t.cuda() for t in W.qkv(w, 0, 0, 0, 0))
    out = [torch.empty_like(q) for _ in range(2)]
    items = [dict(stage=0, chunk_index=i, n_frames=1, first_frame_pos=i, q=q.data_ptr(), k=k.data_ptr(), v=v.data_ptr(),
                  out=out[i].data_ptr(), anchor_slots=[]) for i in range(2)]
    assert gpu.cache.ff_batch_forward_attn(0, items, gpu.stream) == gpu.P.FF_ERR_UNSUPPORTED
    assert gpu.cache.ff_batch_forward_attn(0, items[::-1], gpu.stream) == gpu.P.FF_ERR_STATE   # out of order
    assert gpu.cache.ff_cache_counters()["layer_calls"] == 0
    gpu.close()
