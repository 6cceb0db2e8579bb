"""The allocation-free entry point against the regular one.

ff_chunk_attn_static serves callers that get device buffers handed to them but must not allocate device memory
themselves (a plug-in inside a server whose pool belongs to the framework, a loop that cannot take cudaMalloc's
implicit synchronisation).  Its scratch is one fixed device array inside the library, shared by all calls, which
still holds the previous call's data when the next call starts - so the check runs two different calls back to
back and compares each (a) with the CPU oracle's first-chunk call (chunk 0, empty bank, no anchors), every row,
within the tolerance of the other parity tests, and (b) with ff_chunk_forward_attn on a fresh cache (CUDA-core
kernel), which computes the same thing out of a caller-provided arena.  A third check reads the device's free
memory around a warm call: the call must not change it.

Collected last on purpose: a failure here cannot hide the result of any other test in a run that stops at the
first failure.  It passes alone in a fresh process and after the other tests.
"""
import pytest
import torch

import ff_workloads as W
from oracle import ff_oracle as O
from tests import ff_harness as Hn

pytestmark = pytest.mark.gpu


def _reference(w, dtype, q, k, v, first_frame_pos):
    gpu = Hn.GpuCache(w, dtype, attn_impl=2)
    st, out = gpu.forward(0, 0, 0, w.chunk_frames, first_frame_pos, q, k, v, [])
    assert st == 0
    torch.cuda.synchronize()
    out = out.clone()
    gpu.close()
    return out


@pytest.mark.parametrize("dtype", [O.BF16, O.F32])
def test_static_scratch_entry_point_matches_arena_entry_point_twice(dtype):
    from paper_2609_32540_b200 import binding as B
    assert torch.cuda.is_available()
    dt = Hn.tdtype(dtype)
    stream = torch.cuda.current_stream().cuda_stream
    # two calls of different shape in a row, so the second one finds the first one's data in the scratch
    cases = [
        (W.Workload("na1", 1, 4, 128, 12, 16, 2, 1, 0, 2, 0, 0, "none", 1), 5, 7),    # 384 tokens: 3 full tiles
        (W.Workload("na2", 1, 2, 64, 9, 11, 1, 1, 0, 1, 0, 0, "none", 1), 6, 0),      # 99 tokens: ragged, smaller
    ]
    for w, seed, pos in cases:
        q, k, v = (t.cuda() for t in W.qkv(w, seed, 0, 0, 0, w.chunk_frames, dt))
        out = torch.full_like(q, float("nan"))
        st = B.ff_chunk_attn_static(w.n_heads, w.head_dim, w.grid_h, w.grid_w, w.chunk_frames, pos, w.rope_theta,
                                    dtype, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), stream)
        assert st == B.FF_OK, st
        torch.cuda.synchronize()
        # (a) the oracle, written from the definition: rotate, publish, attend over the chunk's own keys
        orc = Hn.make_oracle(w, dtype)
        so, truth = orc.chunk_forward(0, 0, 0, w.chunk_frames, pos, q.float().cpu().numpy(), k.float().cpu().numpy(),
                                      v.float().cpu().numpy(), [])
        assert so == O.OK
        Hn.compare_outputs(out, truth, dtype, f"static entry point, {w.name}")
        # (b) the arena entry point: same kernels; its rotary tables are evaluated on the host, this one's on the
        # device, so a rotated element may differ in its last bit
        want = _reference(w, dtype, q, k, v, pos)
        err = (out.float() - want.float()).abs()
        tol = Hn.F32_ABS_TOL if dtype == O.F32 else Hn.ABS_MAX_TOL
        assert err.max().item() <= tol, err.max().item()


def test_static_scratch_entry_point_leaves_free_device_memory_unchanged():
    """The claim "allocates nothing", measured: free device memory before and after a call on a warm library (the
    first call on a device may load the kernels' module) is the same to the byte."""
    from paper_2609_32540_b200 import binding as B
    w = W.Workload("na3", 1, 2, 64, 8, 8, 1, 1, 0, 1, 0, 0, "none", 1)
    q, k, v = (t.cuda() for t in W.qkv(w, 3, 0, 0, 0, 1, torch.bfloat16))
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        assert B.ff_chunk_attn_static(w.n_heads, w.head_dim, w.grid_h, w.grid_w, 1, 0, w.rope_theta, B.FF_BF16,
                                      q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), stream) == B.FF_OK
        torch.cuda.synchronize()

    call()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        call()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    from paper_2609_32540_b200 import binding as B
    # 3 * 4736 rows * 12 heads * 128 * 2 B = 43.6 MB > 8 MiB
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    st = B.ff_chunk_attn_static(12, 128, 30, 52, 3, 0, 10000.0, B.FF_BF16, x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                x.data_ptr(), 0)
    assert st == B.FF_ERR_OOM
    assert B.ff_chunk_attn_static(2, 96, 4, 4, 1, 0, 10000.0, B.FF_BF16, x.data_ptr(), x.data_ptr(), x.data_ptr(),
                                  x.data_ptr(), 0) == B.FF_ERR_UNSUPPORTED
