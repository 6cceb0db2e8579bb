"""Seeded random small configurations through all three schedules (chunk-major, wavefront rounds, clip at once):
shapes chosen to hit ragged tiles, single-tile chunks, short last chunks, empty anchor lists, H = 0 and the
work-distribution corner cases (fewer pairs than SMs, one key tile, cut pairs across items), on all three
attention kernels."""
import random

import pytest
import torch

import ff_workloads as W
from oracle import ff_oracle as O
from tests import ff_harness as Hn

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2609_32540_b200 import binding
    binding.load()   # fails loudly when the extension is missing


def _random_workload(seed: int) -> W.Workload:
    r = random.Random(seed)
    head_dim = r.choice([64, 128])
    n_heads = r.choice([1, 2, 3, 5])
    grid_h, grid_w = r.randint(3, 14), r.randint(3, 17)
    chunk_frames = r.choice([1, 2, 3])
    n_stages = r.choice([1, 2, 3, 4])
    H = r.choice([0, 1, 2, 3])
    n_chunks = r.randint(2, 6)
    short_last = r.random() < 0.5 and chunk_frames > 1
    total_frames = n_chunks * chunk_frames - (r.randint(1, chunk_frames - 1) if short_last else 0)
    policy = r.choice(["none", "ahead", "every", "bracket"])
    period = r.randint(2, 6)
    vis = 0 if policy == "none" else (2 if policy == "bracket" else 1)
    n_slots = 0 if policy == "none" else total_frames // period + 3      # one slot per anchor: valid in every schedule
    return W.Workload(f"random{seed}", r.choice([1, 2]), n_heads, head_dim, grid_h, grid_w, chunk_frames, n_stages, H,
                      total_frames, vis, n_slots, policy, period, max_frame_pos=256)


@pytest.mark.parametrize("seed", list(range(32)))
def test_random_configuration_in_all_three_schedules(seed):
    w = _random_workload(seed)
    rows = None if w.chunk_frames * w.tokens_per_frame <= 400 else (lambda n: W.sample_rows(n, 24, seed))
    # every fifth seed runs the fp32 cache on the CUDA-core kernel instead of bf16 on a tensor-core kernel; of the
    # others, those with head_dim 128 alternate between the one-CTA-per-SM kernel (1) and the kernel on CTA pairs (3)
    dtype, impl = (O.F32, 2) if seed % 5 == 4 else (O.BF16, 3 if w.head_dim == 128 and seed % 2 == 0 else 1)
    stats, gpu, _ = Hn.run_both(w, dtype, attn_impl=impl, seed=seed, rows_fn=rows)
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()
    stats, gpu, _ = Hn.run_wavefront(w, dtype, attn_impl=impl, seed=seed, rows_fn=rows, use_round_call=seed % 2 == 0)
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()
    group = 1 + seed % 4
    stats, gpu, _ = Hn.run_packed_clip(w, group, dtype, attn_impl=impl, seed=seed, rows_fn=rows)
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()


@pytest.mark.parametrize("seed", list(range(100, 116)))
def test_random_configuration_with_the_fused_qk_normalisation(seed):
    """The same kind of shapes with raw Q/K rows and the normalisation fused into the publish pass (every other
    seed with per-channel gains): the published cache must still match the oracle bit for bit."""
    w = _random_workload(seed)
    rows = None if w.chunk_frames * w.tokens_per_frame <= 400 else (lambda n: W.sample_rows(n, 24, seed))
    dtype, impl = (O.F32, 2) if seed % 5 == 4 else (O.BF16, 3 if w.head_dim == 128 and seed % 2 == 0 else 1)
    stats, gpu, _ = Hn.run_both(w, dtype, attn_impl=impl, seed=seed, rows_fn=rows, qk_norm_eps=1e-6,
                                qk_gains=(seed % 2 == 0))
    assert len(stats) == w.n_chunks * w.n_stages * w.n_layers
    gpu.close()
