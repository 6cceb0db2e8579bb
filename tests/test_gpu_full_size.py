"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: every layer and stage runs
on the GPU; the CPU oracle follows a few (stage, layer) pairs, computes sampled query rows one by one (tile
edges, the ragged tail, seeded others) and compares the published cache slots in full, bit for bit."""
import pytest
import torch

import ff_workloads as W
from oracle import ff_oracle as O
from tests import ff_harness as Hn

pytestmark = pytest.mark.gpu


def rows_fn(n_q):
    return W.sample_rows(n_q, extra=6)


def test_wan1p3b_480p_full_shape():
    """Config 2: 30 layers, 12 heads, d 128, 4680 query tokens, N_kv up to 15600; warm-up chunks, steady state
    and the switch to the second anchor slot (chunk 4)."""
    w = W.scaled(W.CONFIGS["wan1p3b_480p"], total_frames=15)
    stats, gpu, orc = Hn.run_both(w, O.BF16, attn_impl=1, seed=2, rows_fn=rows_fn, check_layers=[0, 29],
                                  check_stages=[0, 3], pooled=True)
    assert len(stats) == 5 * 2 * 2
    c = gpu.cache.ff_cache_counters()
    assert c["layer_calls"] == 5 * 4 * 30 and c["advances"] == 5 * 4 and c["anchor_publishes"] == 2 * 30
    gpu.close()


@pytest.mark.parametrize("name,frames,layer", [("wan1p3b_480p", 12, 1), ("wan1p3b_720p", 9, 0)])
def test_cta_pair_kernel_at_full_token_counts(name, frames, layer):
    """The kernel on CTA pairs (cta_group::2), forced: 480p (37 query tiles per head: the last unit of a head holds
    one tile of four) and 720p (85 tiles), warm-up and steady-state chunks, sampled rows and published slots."""
    w = W.scaled(W.CONFIGS[name], total_frames=frames, n_layers=2)
    stats, gpu, orc = Hn.run_both(w, O.BF16, attn_impl=3, seed=12, rows_fn=rows_fn, check_layers=[layer],
                                  check_stages=[0, 2], pooled=True)
    assert len(stats) == (frames // 3) * 2
    gpu.close()


def test_wan1p3b_480p_every_row_of_a_steady_state_call():
    """One steady-state layer-call of config 2 (anchor + two history chunks + own chunk: 15600 keys) compared with
    the oracle on ALL 4680 rows x 12 heads, not a sample: about half a minute of CPU work for the oracle."""
    w = W.scaled(W.CONFIGS["wan1p3b_480p"], total_frames=9, n_layers=1)
    stats, gpu, orc = Hn.run_both(w, O.BF16, attn_impl=0, seed=11, rows_fn=None, check_layers=[0], check_stages=[1],
                                  pooled=True, check_chunks=[2])
    assert len(stats) == 1 and stats[0]["max_abs"] > 0
    gpu.close()


def test_wan1p3b_480p_peaked_logits():
    """Same shape with logits x8: O(1) outputs, so a dropped segment or tile cannot hide under the tolerance."""
    w = W.scaled(W.CONFIGS["wan1p3b_480p"], total_frames=9, n_layers=2)
    stats, gpu, orc = Hn.run_both(w, O.BF16, attn_impl=1, seed=4, rows_fn=rows_fn, check_layers=[1],
                                  check_stages=[2], pooled=True, logit_gain=8.0)
    assert len(stats) == 3
    gpu.close()


def test_wan1p3b_720p_full_shape():
    """Config 4: 10800 query tokens, two anchor frames, N_kv up to 39600."""
    w = W.scaled(W.CONFIGS["wan1p3b_720p"], total_frames=12)
    stats, gpu, orc = Hn.run_both(w, O.BF16, attn_impl=0, seed=5, rows_fn=rows_fn, check_layers=[17],
                                  check_stages=[1], pooled=True, check_chunks=[0, 3])
    assert len(stats) == 2
    gpu.close()


def test_wan14b_720p_full_shape():
    """Config 5: 40 layers x 40 heads (117 GB arena); one followed (stage, layer), first and steady-state chunk."""
    w = W.scaled(W.CONFIGS["wan14b_720p_stream35s"], total_frames=9)
    free, total = torch.cuda.mem_get_info()
    assert free > 130e9, f"needs about 120 GB of free device memory, have {free / 1e9:.0f} GB"
    stats, gpu, orc = Hn.run_both(w, O.BF16, attn_impl=0, seed=6, rows_fn=lambda n: W.sample_rows(n, extra=2),
                                  check_layers=[39], check_stages=[3], pooled=True, check_chunks=[0, 2])
    assert len(stats) == 2
    gpu.close()
    torch.cuda.empty_cache()


def test_wan1p3b_480p_long_stream():
    """Config 3: the 261-frame stream (87 chunks, 22 anchor publishes, ring and anchor-slot reuse throughout) with
    all 4 stages and all 30 layers on one GPU; the oracle follows one (stage, layer) through the whole stream and compares outputs
    at the start, in the middle and at the end, and the published slot at those chunks."""
    w = W.CONFIGS["wan1p3b_480p_stream65s"]
    assert w.n_chunks == 87 and w.n_layers == 30
    stats, gpu, orc = Hn.run_both(w, O.BF16, attn_impl=1, seed=7, rows_fn=lambda n: W.sample_rows(n, extra=2),
                                  check_layers=[29], check_stages=[0], pooled=True, check_chunks=[0, 1, 2, 3, 4, 43, 85, 86])
    assert len(stats) == 8
    c = gpu.cache.ff_cache_counters()
    assert c["layer_calls"] == 87 * 4 * 30 and c["advances"] == 87 * 4 and c["anchor_publishes"] == 22 * 30
    for stage in range(4):
        s = gpu.cache.ff_cache_ring_state(stage, 0)
        assert s["next_chunk"] == 87 and s["head"] == 87 % 3 and s["count"] == 2
        assert sorted(s["slot_chunk"]) == [84, 85, 86]
    gpu.close()


@pytest.mark.parametrize("name,chunks", [("wan1p3b_480p", 5), ("wan1p3b_720p", 4)])
def test_every_row_at_full_token_counts_agrees_between_the_two_tensor_core_kernels(name, chunks):
    """An extra next to the sampled-row comparisons with the oracle (CUDA against CUDA, so it pins nothing by
    itself): over warm-up and steady-state chunks at full token counts, EVERY output row of the kernel with one
    CTA per SM and of the kernel on CTA pairs is finite and the two agree to a bf16 rounding step.  Their work
    distributions differ (pairs of tiles against units of four, other cut points), so a row that one of them
    dropped or merged wrongly cannot hide here."""
    from tests import test_gpu_api as A
    base = W.CONFIGS[name]
    w = W.scaled(base, n_layers=1, n_stages=1, total_frames=chunks * base.chunk_frames)
    a, ga = A._run(w, "chunk", impl=1)
    b, gb = A._run(w, "chunk", impl=3)
    assert len(a) == chunks
    for key in a:
        assert torch.isfinite(a[key].float()).all() and torch.isfinite(b[key].float()).all(), key
        worst = (a[key].float() - b[key].float()).abs().max().item()
        assert worst <= 2e-3, (key, worst)
    ga.close(); gb.close()
