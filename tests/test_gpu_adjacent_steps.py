"""The steps next to the chunk-attention path, on a B200 through the C ABI: the q/k normalisation fused into the
publish pass, and the Euler update that follows a forward (Alg. 1, "Step")."""
import numpy as np
import pytest
import torch

import ff_workloads as W
from oracle import ff_oracle as O
from oracle import paper_defs as PD
from tests import ff_harness as Hn

pytestmark = pytest.mark.gpu

TINY = W.CONFIGS["tiny"]


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2609_32540_b200 import binding
    binding.load()   # fails loudly when the extension is missing


@pytest.mark.parametrize("dtype,impl", [(O.F32, 2), (O.BF16, 2), (O.BF16, 1)])
def test_fused_qk_norm_tiny_stream(dtype, impl):
    """Raw rows whose magnitudes spread over two decades go in; the published K' must equal the oracle's bit for
    bit (same order of every rounding), the outputs within the usual tolerance; anchors take the same route."""
    stats, gpu, orc = Hn.run_both(TINY, dtype, attn_impl=impl, seed=2, qk_norm_eps=1e-6, qk_gains=True)
    assert len(stats) == TINY.n_chunks * TINY.n_stages * TINY.n_layers
    gpu.close()


def test_fused_qk_norm_head_dim_128_ragged_multi_tile():
    """d = 128 (16 pieces per row in bf16), several heads, a token count that is not a multiple of the tile, a
    short last chunk, two anchors in the window."""
    w = W.Workload("norm_ragged", 2, 3, 128, 9, 23, 2, 2, 2, 7, 2, 3, "bracket", 4)
    stats, gpu, orc = Hn.run_both(w, O.BF16, attn_impl=1, seed=4, qk_norm_eps=1e-6, qk_gains=True,
                                  rows_fn=lambda n: W.sample_rows(n, 24, 1))
    assert stats and max(s["max_abs"] for s in stats) <= Hn.ABS_MAX_TOL
    gpu.close()


def test_fused_qk_norm_cache_is_within_one_bf16_ulp_of_the_float64_definition():
    """The bit-exact comparisons above rest on the oracle summing squares in the same order as the kernel (running
    sums over 16-byte pieces, then a balanced tree).  This one does not: the published K' is compared with
    normalise -> gain -> rotate written out in float64 here (numpy for the normalisation, the complex-form rotary
    of the paper definitions), and must agree to one bf16 unit in the last place."""
    w = W.Workload("norm_f64", 1, 3, 128, 5, 9, 2, 1, 1, 2, 0, 0, "none", 1)
    eps = 1e-6
    gpu = Hn.GpuCache(w, O.BF16, attn_impl=1, qk_norm_eps=eps)
    gq, gk = W.channel_gains(w, 13, 0)
    assert gpu.cache.ff_cache_set_qk_gain(0, gq.tolist(), gk.tolist(), gpu.stream) == 0
    q, k, v = W.qkv(w, 13, 0, 0, 0, w.chunk_frames, torch.bfloat16, pre_normalised=False)
    st, out = gpu.forward(0, 0, 0, w.chunk_frames, 3, q.cuda(), k.cuda(), v.cuda(), [])
    assert st == 0
    torch.cuda.synchronize()
    n = k.shape[0]
    ck, cv, _ = gpu.read_slot(0, 0, 0, 0, n)
    x = k.double().numpy()
    normed = x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * gk.double().numpy()
    want = PD.rope_complex(normed, PD.token_positions(w.chunk_frames, 3, w.grid_h, w.grid_w)[:, None, :])
    got = ck.double().numpy()
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 2.0 ** -126))) - 7)     # bf16: 8 significant bits
    assert np.all(np.abs(got - want) <= ulp), float((np.abs(got - want) / ulp).max())
    assert np.array_equal(Hn.bits(cv), Hn.bits(v))
    gpu.close()


def test_qk_norm_off_rejects_gain_and_unit_gain_equals_no_gain():
    gpu = Hn.GpuCache(TINY, O.BF16)
    assert gpu.cache.ff_cache_set_qk_gain(0, [1.0] * TINY.head_dim, None, gpu.stream) == gpu.P.FF_ERR_STATE
    gpu.close()
    on = Hn.GpuCache(TINY, O.BF16, qk_norm_eps=1e-6)
    assert on.cache.ff_cache_set_qk_gain(0, None, None, on.stream) == on.P.FF_ERR_INVALID_ARG
    assert on.cache.ff_cache_set_qk_gain(TINY.n_layers, [1.0] * TINY.head_dim, None, on.stream) == on.P.FF_ERR_INVALID_ARG
    on.close()


@pytest.mark.parametrize("dx,dv", [(torch.float32, torch.bfloat16), (torch.float32, torch.float32),
                                   (torch.bfloat16, torch.bfloat16), (torch.bfloat16, torch.float32)])
@pytest.mark.parametrize("n", [0, 1, 7, 8, 4099, 299520, 148 * 8 * 256 * 8 + 13])
def test_euler_step_bit_exact(n, dx, dv):
    import paper_2609_32540_b200 as P
    code = {torch.float32: P.FF_F32, torch.bfloat16: P.FF_BF16}
    x, v = W.latent_and_velocity(max(n, 1), 5, 0, 3, dx, dv)
    x, v = x[:n], v[:n]
    sig = PD.sigma_schedule(4, 5.0)
    want = O.euler_step(x.float().numpy(), v.float().numpy(), np.float32(sig[3]), np.float32(sig[2]),
                        round_bf16=dx == torch.bfloat16)
    xd = torch.zeros(n + 16, dtype=dx, device="cuda")
    vd = torch.zeros(n + 16, dtype=dv, device="cuda")
    xd[:n], vd[:n] = x.cuda(), v.cuda()
    out = torch.full((n + 16,), 7.0, dtype=dx, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    assert P.ff_euler_step(xd.data_ptr(), vd.data_ptr(), sig[3], sig[2], n, code[dx], code[dv], out.data_ptr(), s) == 0
    torch.cuda.synchronize()
    assert np.array_equal(Hn.bits(out[:n].cpu()), Hn.bits(torch.from_numpy(want).to(dx)))
    assert bool((out[n:] == 7.0).all()), "wrote past n"
    # in place
    assert P.ff_euler_step(xd.data_ptr(), vd.data_ptr(), sig[3], sig[2], n, code[dx], code[dv], xd.data_ptr(), s) == 0
    torch.cuda.synchronize()
    assert np.array_equal(Hn.bits(xd[:n].cpu()), Hn.bits(torch.from_numpy(want).to(dx)))


def test_euler_step_walks_the_library_schedule_to_the_clean_latent():
    """sigma from ff_plan_sigma, exact velocity: four updates take pure noise to x0."""
    import paper_2609_32540_b200 as P
    n = 299520   # one 480p chunk of latents: 3 frames x 16 channels x 60 x 104
    x0, eps = W.latent_and_velocity(n, 9, 1, 0, torch.float32, torch.float32)
    v = (eps - x0).cuda()
    x = eps.clone().cuda()
    s = torch.cuda.current_stream().cuda_stream
    sig = [P.ff_plan_sigma(k, 4, 5.0) for k in range(5)]
    assert sig == PD.sigma_schedule(4, 5.0)
    for k in range(4, 0, -1):
        assert P.ff_euler_step(x.data_ptr(), v.data_ptr(), sig[k], sig[k - 1], n, P.FF_F32, P.FF_F32, x.data_ptr(), s) == 0
    torch.cuda.synchronize()
    assert float((x.cpu() - x0).abs().max()) < 5e-6


def test_euler_step_argument_errors():
    import paper_2609_32540_b200 as P
    x = torch.zeros(64, device="cuda")
    p = x.data_ptr()
    assert P.ff_euler_step(0, p, 1.0, 0.5, 8, P.FF_F32, P.FF_F32, p, 0) == P.FF_ERR_INVALID_ARG
    assert P.ff_euler_step(p + 4, p, 1.0, 0.5, 8, P.FF_F32, P.FF_F32, p, 0) == P.FF_ERR_INVALID_ARG
    assert P.ff_euler_step(p, p, 1.0, 0.5, -1, P.FF_F32, P.FF_F32, p, 0) == P.FF_ERR_INVALID_ARG
    assert P.ff_euler_step(p, p, float("nan"), 0.5, 8, P.FF_F32, P.FF_F32, p, 0) == P.FF_ERR_INVALID_ARG
    assert P.ff_euler_step(p, p, 1.0, 0.5, 8, 5, P.FF_F32, p, 0) == P.FF_ERR_INVALID_ARG


def test_one_rank_wavefront_drives_attention_and_euler_on_the_gpu():
    """The stage-per-rank driver with a single stage (so no message leaves the rank): every chunk's node runs all
    layers through the library's cache and then the Euler update; attention outputs and the delivered latents are
    compared with the oracle."""
    import paper_2609_32540_b200 as P
    from paper_2609_32540_b200 import wavefront as Wf
    w = W.scaled(TINY, anchor_policy="none", n_anchor_slots=0, n_stages=1, n_layers=2)
    gpu = Hn.GpuCache(w, O.BF16, attn_impl=1)
    orc = Hn.make_oracle(w, O.BF16)
    sig = [P.ff_plan_sigma(k, 1, 5.0) for k in range(2)]          # one stage: sigma_1 = 1 -> sigma_0 = 0
    n_lat = 1000
    delivered, checked = {}, []

    def run_node(i, x):
        io_t = []
        for l in range(w.n_layers):
            q, k, v = (t.cuda() for t in W.qkv(w, 31, i, 0, l))
            io_t.append((q, k, v, torch.full_like(q, float("nan"))))
        io = P.make_io([(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr()) for q, k, v, o in io_t])
        assert gpu.cache.ff_sched_run_node(0, i, 1, i, [], io, gpu.stream) == 0
        _, vhat = W.latent_and_velocity(n_lat, 31, i, 0, torch.float32, torch.bfloat16)
        vd = vhat.cuda()
        y = torch.empty_like(x)
        assert P.ff_euler_step(x.data_ptr(), vd.data_ptr(), sig[1], sig[0], n_lat, P.FF_F32, P.FF_BF16, y.data_ptr(), gpu.stream) == 0
        torch.cuda.synchronize()
        for l, (q, k, v, o) in enumerate(io_t):
            so, want = orc.chunk_forward(0, l, i, 1, i, q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy())
            assert so == 0
            checked.append(Hn.compare_outputs(o, want, O.BF16, f"chunk {i} layer {l}"))
        assert orc.advance(0) == 0
        return y

    like = torch.zeros(n_lat, dtype=torch.float32, device="cuda")
    sr = Wf.StageRank(0, 1, w.n_chunks, like,
                      obtain=lambda i: W.latent_and_velocity(n_lat, 31, i, 0, torch.float32, torch.bfloat16)[0].cuda(),
                      run_node=run_node, deliver=lambda i, x: delivered.__setitem__(i, x.cpu()))
    stats = sr.run()
    assert stats.chunks == w.n_chunks and stats.sent == 0 and stats.received == 0
    assert len(checked) == w.n_chunks * w.n_layers and sorted(delivered) == list(range(w.n_chunks))
    for i in range(w.n_chunks):
        x, vhat = W.latent_and_velocity(n_lat, 31, i, 0, torch.float32, torch.bfloat16)
        want = O.euler_step(x.numpy(), vhat.float().numpy(), np.float32(sig[1]), np.float32(sig[0]))
        assert np.array_equal(delivered[i].numpy(), want)
    gpu.close()
