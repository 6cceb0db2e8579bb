"""Pins of the CPU oracle against things other than itself: the textbook softmax in float64, a library
attention routine, closed-form invariants, rotation identities, the packed full-clip formulation, and
isolation of everything outside the visible set."""
import math

import numpy as np
import pytest
import torch

import ff_workloads as W
from oracle import ff_oracle as O
from oracle import paper_defs as P

TINY = W.CONFIGS["tiny"]


def make_oracle(w, dtype=O.BF16, **kw):
    args = dict(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
                chunk_frames=w.chunk_frames, n_stages=w.n_stages, history_chunks=w.history_chunks,
                n_anchor_slots=w.n_anchor_slots, dtype=dtype, rope_theta=w.rope_theta)
    args.update(kw)
    return O.Oracle(**args)


def tdtype(dtype):
    return torch.bfloat16 if dtype == O.BF16 else torch.float32


def run_stream(w, orc, dtype, seed=0, n_chunks=None, logit_gain=1.0, record=None):
    """Chunk-major stream through the oracle; returns {(chunk, stage, layer): out}."""
    outs = {}
    for ev in W.trace(w, n_chunks):
        if ev.kind == "anchor":
            for l in range(w.n_layers):
                k, v = W.anchor_kv(w, seed, ev.anchor_id, l, tdtype(dtype))
                assert orc.anchor_publish(ev.slot, ev.frame_pos, l, k.float().numpy(), v.float().numpy()) == O.OK
                if record is not None:
                    record.setdefault("anchors", {})[(ev.anchor_id, l)] = (k, v, ev.frame_pos)
            continue
        for stage in reversed(range(w.n_stages)):
            for l in range(w.n_layers):
                q, k, v = W.qkv(w, seed, ev.chunk, stage, l, ev.n_frames, tdtype(dtype), logit_gain)
                st, out = orc.chunk_forward(stage, l, ev.chunk, ev.n_frames, ev.first_frame_pos, q.float().numpy(),
                                            k.float().numpy(), v.float().numpy(), ev.anchor_slots)
                assert st == O.OK
                outs[(ev.chunk, stage, l)] = out
                if record is not None:
                    record.setdefault("calls", {})[(ev.chunk, stage, l)] = (q, k, v, ev)
            assert orc.advance(stage) == O.OK
    return outs


# ----------------------------------------------------------------------------- bf16 rounding

def test_bf16_round_matches_library_cast():
    g = torch.Generator().manual_seed(1)
    x = torch.randn(4096, generator=g) * torch.logspace(-20, 20, 4096)
    # ties: values exactly halfway between two bf16 neighbours
    ties = torch.tensor([1.00390625, 1.01171875, -3.0078125, 2.0 ** -126 * 1.00390625])
    x = torch.cat([x, ties])
    want = x.to(torch.bfloat16).float().numpy()
    got = O.bf16_round(x.numpy())
    assert np.array_equal(want.view(np.uint32), got.view(np.uint32))


# ----------------------------------------------------------------------------- rotary identities (step 1)

@pytest.mark.parametrize("d", [64, 128])
def test_rope_identity_at_origin_and_norm_preserved(d):
    rng = np.random.default_rng(0)
    x = rng.standard_normal(d).astype(np.float32)
    assert np.array_equal(O.rope_vec(x, (0, 0, 0)), x)
    y = O.rope_vec(x, (37, 29, 51))
    nx = np.hypot(x[0::2], x[1::2])
    ny = np.hypot(y[0::2], y[1::2])
    assert np.allclose(nx, ny, rtol=1e-6, atol=1e-7)
    assert not np.allclose(x, y, atol=1e-3)


@pytest.mark.parametrize("d", [64, 128])
def test_rope_inverse_and_composition(d):
    rng = np.random.default_rng(1)
    x = rng.standard_normal(d).astype(np.float32)
    p = (11, 7, 23)
    back = O.rope_vec(O.rope_vec(x, p), tuple(-a for a in p))
    assert np.allclose(back, x, atol=5e-6)
    # rotating by p1 then p2 equals rotating by p1 + p2
    a = O.rope_vec(O.rope_vec(x, (3, 4, 5)), (8, 3, 18))
    b = O.rope_vec(x, (11, 7, 23))
    assert np.allclose(a, b, atol=5e-6)


def test_rope_axis_groups_and_first_pair_angle():
    d = 128
    n_t, n_h, n_w = O.default_pairs(d)
    assert (n_t, n_h, n_w) == (22, 21, 21) and O.default_pairs(64) == (12, 10, 10)
    e = np.zeros(d, np.float32)
    # pair 0 of each axis group turns by exactly `pos` radians: (1,0) -> (cos pos, sin pos), counter-clockwise
    for axis, m in enumerate((0, n_t, n_t + n_h)):
        x = e.copy()
        x[2 * m] = 1.0
        pos = [0, 0, 0]
        pos[axis] = 2
        y = O.rope_vec(x, pos)
        assert y[2 * m] == np.float32(math.cos(2.0)) and y[2 * m + 1] == np.float32(math.sin(2.0))
        # a position on another axis leaves this pair alone
        other = [5, 5, 5]
        other[axis] = 0
        assert np.array_equal(O.rope_vec(x, other), x)
    # within a group the turn angle decreases with the pair index (geometric frequencies, last one > 1/theta)
    x = np.zeros(d, np.float32)
    x[0:2 * n_t:2] = 1.0
    y = O.rope_vec(x, (1, 0, 0))
    ang = np.arctan2(y[1:2 * n_t:2], y[0:2 * n_t:2])
    assert np.all(np.diff(ang) < 0) and ang[0] == pytest.approx(1.0, abs=1e-6) and ang[-1] > 1e-4
    ratios = ang[1:] / ang[:-1]
    assert np.allclose(ratios, ratios[0], rtol=1e-3)
    assert ang[-1] * ratios[0] == pytest.approx(1e-4, rel=1e-2)   # one more step would reach 1/theta


def test_rope_matches_complex_form():
    rng = np.random.default_rng(2)
    for d in (64, 128):
        x = rng.standard_normal((5, d)).astype(np.float32)
        pos = np.array([[0, 0, 0], [1, 2, 3], [20, 29, 51], [260, 44, 79], [7, 0, 13]])
        want = P.rope_complex(x, pos)
        got = np.stack([O.rope_vec(x[i], pos[i]) for i in range(5)])
        assert np.allclose(got, want, atol=3e-6)


# ----------------------------------------------------------------------------- step 4 vs textbook definitions

def test_no_history_no_anchor_is_plain_bidirectional_attention_sdpa():
    """Empty bank and no anchors: the call is ordinary attention inside the chunk (a library routine is the referee)."""
    w = W.scaled(TINY, anchor_policy="none", visible_anchors=0)
    orc = make_oracle(w, O.F32)
    q, k, v = W.qkv(w, 3, 0, 0, 0, 1, torch.float32)
    st, out = orc.chunk_forward(0, 0, 0, 1, 0, q.numpy(), k.numpy(), v.numpy())
    assert st == O.OK
    pos = P.token_positions(1, 0, w.grid_h, w.grid_w)[:, None, :]
    qr = torch.from_numpy(P.rope_complex(q.numpy(), pos)).permute(1, 0, 2)
    kr = torch.from_numpy(P.rope_complex(k.numpy(), pos)).permute(1, 0, 2)
    want = torch.nn.functional.scaled_dot_product_attention(qr, kr, v.double().permute(1, 0, 2)).permute(1, 0, 2)
    assert np.allclose(out, want.numpy(), atol=2e-6)


@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_stream_matches_bruteforce_float64(dtype):
    """Every call of the tiny stream against the textbook softmax over an independently gathered key set."""
    w = TINY
    orc = make_oracle(w, dtype)
    rec = {}
    outs = run_stream(w, orc, dtype, seed=0, record=rec)
    H = w.history_chunks
    worst = 0.0
    for (i, stage, l), out in outs.items():
        q, k, v, ev = rec["calls"][(i, stage, l)]
        ks, vs = [], []
        for m in ev.anchor_ids:
            ak, av, fpos = rec["anchors"][(m, l)]
            pos = P.token_positions(1, fpos, w.grid_h, w.grid_w)[:, None, :]
            ks.append(P.rope_complex(ak.float().numpy(), pos))
            vs.append(av.double().numpy())
        for j in range(max(0, i - H), i + 1):
            qj, kj, vj, evj = rec["calls"][(j, stage, l)]
            pos = P.token_positions(evj.n_frames, evj.first_frame_pos, w.grid_h, w.grid_w)[:, None, :]
            ks.append(P.rope_complex(kj.float().numpy(), pos))
            vs.append(vj.double().numpy())
        K, V = np.concatenate(ks), np.concatenate(vs)
        pos = P.token_positions(ev.n_frames, ev.first_frame_pos, w.grid_h, w.grid_w)[:, None, :]
        Q = P.rope_complex(q.float().numpy(), pos)
        for h in range(w.n_heads):
            want = P.softmax_attention(Q[:, h], K[:, h], V[:, h])
            worst = max(worst, float(np.abs(out[:, h] - want).max()))
    # F32: only rounding of the rotation; BF16: Q' and K' are rounded to bf16 before the scores
    assert worst < (2e-5 if dtype == O.F32 else 2e-2), worst
    assert len(outs) == w.n_chunks * w.n_stages * w.n_layers


def test_sequential_bank_equals_packed_block_mask():
    """Updating B_k chunk by chunk equals one full-clip forward under the chunk-wise causal mask, including
    warm-up chunks, a short last chunk and two layers."""
    w = W.scaled(TINY, n_layers=2, chunk_frames=2, total_frames=9, grid_h=3, grid_w=4, n_anchor_slots=4,
                 anchor_period_frames=4)
    orc = make_oracle(w, O.F32)
    rec = {}
    outs = run_stream(w, orc, O.F32, seed=5, record=rec)
    assert w.n_chunks == 5 and w.chunk_frames_of(4) == 1
    for stage in range(w.n_stages):
        for l in range(w.n_layers):
            chunks, vis = [], []
            for i in range(w.n_chunks):
                q, k, v, ev = rec["calls"][(i, stage, l)]
                chunks.append(dict(q=q.numpy(), k=k.numpy(), v=v.numpy(), n_frames=ev.n_frames,
                                   first_frame_pos=ev.first_frame_pos))
                vis.append(ev.anchor_ids)
            anchors = {m: dict(k=ak.numpy(), v=av.numpy(), frame_pos=fp)
                       for (m, ll), (ak, av, fp) in rec["anchors"].items() if ll == l}
            packed = P.packed_block_mask_attention(chunks, anchors, vis, w.history_chunks, w.grid_h, w.grid_w)
            for i in range(w.n_chunks):
                assert np.allclose(outs[(i, stage, l)], packed[i], atol=2e-5), (stage, l, i)


# ----------------------------------------------------------------------------- closed-form invariants

def test_constant_v_returns_v_and_identical_keys_return_mean():
    w = TINY
    for case in ("const_v", "same_k"):
        orc = make_oracle(w, O.BF16)
        for ev in W.trace(w):
            if ev.kind == "anchor":
                k, v = W.anchor_kv(w, 0, ev.anchor_id, 0)
                k, v = k.float().numpy(), v.float().numpy()
                if case == "const_v":
                    v[:] = np.float32(0.75) * np.arange(1, w.head_dim + 1, dtype=np.float32)[None, None, :] / 64
                assert orc.anchor_publish(ev.slot, ev.frame_pos, 0, k, v) == O.OK
                continue
            q, k, v = (t.float().numpy() for t in W.qkv(w, 0, ev.chunk, 0, 0, ev.n_frames))
            if case == "const_v":
                v[:] = np.float32(0.75) * np.arange(1, w.head_dim + 1, dtype=np.float32)[None, None, :] / 64
            st, out = orc.chunk_forward(0, 0, ev.chunk, ev.n_frames, ev.first_frame_pos, q, k, v, ev.anchor_slots)
            assert st == O.OK and orc.advance(0) == O.OK
            if case == "const_v":
                assert np.allclose(out, v[:1], atol=1e-6)
        if case == "same_k":
            # one chunk, no anchors, all keys zero => every score is 0 => uniform weights => mean of V
            orc2 = make_oracle(W.scaled(w, anchor_policy="none"), O.BF16)
            q, k, v = (t.float().numpy() for t in W.qkv(w, 1, 0, 0, 0, 1))
            k[:] = 0.0
            st, out = orc2.chunk_forward(0, 0, 0, 1, 0, q, k, v)
            assert np.allclose(out, v.mean(axis=0, keepdims=True).repeat(len(q), 0), atol=1e-6)


def test_planted_key_dominates():
    """A key equal to (a large multiple of) the query direction at the same position pulls the output to its V row."""
    w = W.scaled(TINY, anchor_policy="none")
    orc = make_oracle(w, O.F32)
    q, k, v = (t.numpy() for t in W.qkv(w, 2, 0, 0, 0, 1, torch.float32))
    k = k.copy()
    k[17] = 40.0 * q[17]      # same token => same rotation => q'.k' = 40 |q|^2 = 40 d
    st, out = orc.chunk_forward(0, 0, 0, 1, 0, q, k, v)
    assert np.allclose(out[17], v[17], atol=1e-4)


# ----------------------------------------------------------------------------- relative positions, permutations

def test_shift_of_all_positions_leaves_output_unchanged():
    w = W.scaled(TINY, anchor_policy="none", n_layers=1, grid_h=4, grid_w=4)
    outs = []
    for shift in (0, 9):
        orc = make_oracle(w, O.F32)
        for i in range(3):
            q, k, v = (t.numpy() for t in W.qkv(w, 4, i, 0, 0, 1, torch.float32))
            st, out = orc.chunk_forward(0, 0, i, 1, i + shift, q, k, v)
            assert st == O.OK and orc.advance(0) == O.OK
        outs.append(out)
    assert np.allclose(outs[0], outs[1], atol=1e-4)
    assert np.abs(outs[0] - outs[1]).max() > 0    # positions do enter the arithmetic


def test_anchor_position_matters_and_may_be_ahead():
    w = W.scaled(TINY, grid_h=4, grid_w=4)
    res = []
    for fpos in (3, 40):
        orc = make_oracle(w, O.F32)
        k, v = (t.numpy() for t in W.anchor_kv(w, 0, 0, 0, torch.float32))
        assert orc.anchor_publish(0, fpos, 0, k, v) == O.OK
        q, kk, vv = (t.numpy() for t in W.qkv(w, 0, 0, 0, 0, 1, torch.float32))
        st, out = orc.chunk_forward(0, 0, 0, 1, 0, q, kk, vv, [0])
        assert st == O.OK
        res.append(out)
    assert np.abs(res[0] - res[1]).max() > 1e-3


def test_token_permutation_inside_a_frame_changes_nothing_but_order():
    """Keys are a set: with the positions taken out of play (a huge rotary base leaves only pair 0 of each axis
    turning, and those input dims are zeroed) permuting the chunk's keys together with their values changes
    nothing."""
    w = W.scaled(TINY, anchor_policy="none", grid_h=1, grid_w=16)
    q, k, v = (t.numpy() for t in W.qkv(w, 6, 0, 0, 0, 1, torch.float32))
    for arr in (q, k):
        arr[..., 0:2] = 0
        arr[..., 24:26] = 0
        arr[..., 44:46] = 0
    orc_a = make_oracle(w, O.F32, rope_theta=1e300)
    st, a = orc_a.chunk_forward(0, 0, 0, 1, 0, q, k, v)
    perm = np.random.default_rng(0).permutation(len(k))
    orc_b = make_oracle(w, O.F32, rope_theta=1e300)
    st, b = orc_b.chunk_forward(0, 0, 0, 1, 0, q, k[perm], v[perm])
    assert np.allclose(a, b, atol=1e-6)


def _strided_positions(n_frames, first, stride, grid_h, grid_w):
    """[n_frames*grid_h*grid_w, 1, 3] positions of a block whose frames sit at first + f*stride (built here, not
    taken from the oracle or from paper_defs.token_positions, which only knows dense chunks)."""
    pos = [(first + f * stride, y, x) for f in range(n_frames) for y in range(grid_h) for x in range(grid_w)]
    return np.asarray(pos, dtype=np.int64)[:, None, :]


def test_order_of_visible_segments_does_not_matter():
    """The visible keys are a set (the licence to read the banks in physical slot order): (a) the oracle, which
    concatenates [anchors | history | own] in that order, equals the textbook softmax over the same keys gathered
    in the opposite order [own | history newest first | anchors reversed]; (b) handing the oracle its anchor
    slots in another order changes the output only by summation rounding."""
    w = W.scaled(TINY, grid_h=3, grid_w=4, n_anchor_slots=2, visible_anchors=2, anchor_policy="none", total_frames=4)
    anchors = {}
    orcs = [make_oracle(w, O.F32) for _ in range(2)]
    for slot, fpos in ((0, 9), (1, 2)):
        k, v = (t.numpy() for t in W.anchor_kv(w, 21, slot, 0, torch.float32))
        anchors[slot] = (k, v, fpos)
        for orc in orcs:
            assert orc.anchor_publish(slot, fpos, 0, k, v) == O.OK
    calls = []
    for i in range(w.n_chunks):
        q, k, v = (t.numpy() for t in W.qkv(w, 21, i, 0, 0, 1, torch.float32))
        calls.append((q, k, v))
        st, out_fwd = orcs[0].chunk_forward(0, 0, i, 1, i, q, k, v, [0, 1])
        st2, out_rev = orcs[1].chunk_forward(0, 0, i, 1, i, q, k, v, [1, 0])
        assert st == O.OK and st2 == O.OK and orcs[0].advance(0) == O.OK and orcs[1].advance(0) == O.OK
        assert np.allclose(out_fwd, out_rev, atol=1e-6)
        ks, vs = [], []
        for j in range(i, max(0, i - w.history_chunks) - 1, -1):          # own first, then history newest first
            pos = P.token_positions(1, j, w.grid_h, w.grid_w)[:, None, :]
            ks.append(P.rope_complex(calls[j][1], pos))
            vs.append(calls[j][2].astype(np.float64))
        for slot in (1, 0):                                               # anchors last, reversed
            ak, av, fpos = anchors[slot]
            ks.append(P.rope_complex(ak, P.token_positions(1, fpos, w.grid_h, w.grid_w)[:, None, :]))
            vs.append(av.astype(np.float64))
        K, V = np.concatenate(ks), np.concatenate(vs)
        Q = P.rope_complex(q, P.token_positions(1, i, w.grid_h, w.grid_w)[:, None, :])
        for h in range(w.n_heads):
            assert np.allclose(out_fwd[:, h], P.softmax_attention(Q[:, h], K[:, h], V[:, h]), atol=2e-5), (i, h)


def test_identical_keys_across_all_segments_return_the_mean_of_all_visible_values():
    """Zero keys in the anchors, in every history chunk and in the own chunk: every score is 0, so the output is
    the plain mean of V over anchor + history + own rows - and only over those (the evicted chunk's values
    must not enter)."""
    w = W.scaled(TINY, grid_h=2, grid_w=4, total_frames=5, anchor_policy="none", n_anchor_slots=2, visible_anchors=2)
    orc = make_oracle(w, O.BF16)
    avs = []
    for slot, fpos in ((0, 7), (1, 3)):
        k, v = (t.float().numpy() for t in W.anchor_kv(w, 33, slot, 0))
        avs.append(v)
        assert orc.anchor_publish(slot, fpos, 0, np.zeros_like(k), v) == O.OK
    vs = []
    for i in range(w.n_chunks):
        q, k, v = (t.float().numpy() for t in W.qkv(w, 33, i, 0, 0, 1))
        vs.append(v)
        st, out = orc.chunk_forward(0, 0, i, 1, i, q, np.zeros_like(k), v, [0, 1])
        assert st == O.OK and orc.advance(0) == O.OK
        visible = np.concatenate(avs + vs[max(0, i - w.history_chunks):i + 1]).astype(np.float64)
        want = visible.mean(axis=0, keepdims=True).repeat(len(q), 0)
        assert np.allclose(out, want, atol=1e-6), i
        if i > w.history_chunks:   # the chunk that left the window would have moved the mean
            with_evicted = np.concatenate(avs + vs[i - w.history_chunks - 1:i + 1]).astype(np.float64).mean(axis=0)
            assert np.abs(with_evicted - want[0]).max() > 1e-3


# ----------------------------------------------------------------------------- planner side (Alg. 1 Phase A)

def _planner_workload():
    # blocks of B_P = 3 anchor latents that lie Delta = 10 positions apart, H_P = 6 earlier blocks visible
    return W.scaled(W.PAPER_480P_PLANNER, n_layers=1, n_heads=2, head_dim=64, grid_h=2, grid_w=3)


@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_planner_blocks_sit_at_the_anchor_positions_of_the_worked_example(dtype):
    """Blocks of anchor latents (frame f of block j at 30 j + 10 f: the worked example's {0,10,20}, {30,40,50},
    {60,70,80}) through an oracle with frame stride 10, every call against the textbook softmax over keys
    rotated at positions written out here."""
    import json, os
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))["worked_example"]
    w = _planner_workload()
    delta = w.frame_pos_stride
    assert delta == gold["delta"] == 10 and w.chunk_frames == gold["B_P"] == 3
    orc = make_oracle(w, dtype, frame_pos_stride=delta)
    blocks = []
    worst = 0.0
    for j in range(3):
        first = j * w.chunk_frames * delta
        frames = [first + f * delta for f in range(w.chunk_frames)]
        assert frames == gold["anchor_positions"][3 * j:3 * j + 3]
        q, k, v = W.qkv(w, 11, j, 0, 0, w.chunk_frames, tdtype(dtype))
        st, out = orc.chunk_forward(0, 0, j, w.chunk_frames, first, q.float().numpy(), k.float().numpy(),
                                    v.float().numpy())
        assert st == O.OK and orc.advance(0) == O.OK
        pos = _strided_positions(w.chunk_frames, first, delta, w.grid_h, w.grid_w)
        blocks.append((P.rope_complex(k.float().numpy(), pos), v.double().numpy()))
        K = np.concatenate([b[0] for b in blocks])
        V = np.concatenate([b[1] for b in blocks])
        Q = P.rope_complex(q.float().numpy(), pos)
        for h in range(w.n_heads):
            want = P.softmax_attention(Q[:, h], K[:, h], V[:, h])
            worst = max(worst, float(np.abs(out[:, h] - want).max()))
        # the bank holds K rotated at the strided positions (a dense-chunk rotation would differ from frame 1 on)
        ck, _ = orc.ring_slot(0, 0, j % (w.history_chunks + 1))
        tol = 1e-5 if dtype == O.F32 else 2.0 ** -7
        assert np.abs(ck - blocks[-1][0]).max() < tol
        dense = P.rope_complex(k.float().numpy(), P.token_positions(w.chunk_frames, first, w.grid_h, w.grid_w)[:, None, :])
        assert np.abs(ck - dense).max() > 0.1
    assert worst < (2e-5 if dtype == O.F32 else 2e-2), worst


def test_planner_republish_keeps_the_clean_endpoint_forward_and_never_reads_the_own_block_twice():
    """Alg. 1 Phase A: S denoising forwards of block j, then one clean-endpoint forward whose K/V are what the
    bank keeps.  Every one of the S+1 calls reads Tail_{H_P}(A) plus its OWN K/V (not the K/V an earlier forward of
    the same block left in the slot), and after the last call the slot holds exactly that call's K'/V."""
    w = _planner_workload()
    S, delta = 4, w.frame_pos_stride
    orc = make_oracle(w, O.F32, frame_pos_stride=delta)
    kept = []      # per finished block: (rotated K of the clean-endpoint forward, its V)
    for j in range(3):
        first = j * w.chunk_frames * delta
        pos = _strided_positions(w.chunk_frames, first, delta, w.grid_h, w.grid_w)
        for f in range(S + 1):
            q, k, v = (t.numpy() for t in W.qkv(w, 12, j, f, 0, w.chunk_frames, torch.float32))
            st, out = orc.chunk_forward(0, 0, j, w.chunk_frames, first, q, k, v)
            assert st == O.OK
            own = (P.rope_complex(k, pos), v.astype(np.float64))
            hist = kept[max(0, j - w.history_chunks):]
            K = np.concatenate([b[0] for b in hist] + [own[0]])
            V = np.concatenate([b[1] for b in hist] + [own[1]])
            Q = P.rope_complex(q, pos)
            for h in range(w.n_heads):
                assert np.allclose(out[:, h], P.softmax_attention(Q[:, h], K[:, h], V[:, h]), atol=2e-5), (j, f, h)
            ck, cv = orc.ring_slot(0, 0, j % (w.history_chunks + 1))
            assert np.array_equal(cv, v) and np.abs(ck - own[0]).max() < 1e-5
            assert orc.ring_state(0)["next_chunk"] == j      # still the same block until Tail is applied
        kept.append(own)
        assert orc.advance(0) == O.OK
        # bit for bit: the slot equals a fresh oracle's publish of the last forward alone
        solo = make_oracle(w, O.F32, frame_pos_stride=delta)
        for jj in range(j):
            z = np.zeros_like(k)
            assert solo.chunk_forward(0, 0, jj, w.chunk_frames, 0, z, z, z, rows=[])[0] == O.OK and solo.advance(0) == O.OK
        assert solo.chunk_forward(0, 0, j, w.chunk_frames, first, q, k, v, rows=[])[0] == O.OK
        a, b = orc.ring_slot(0, 0, j % (w.history_chunks + 1)), solo.ring_slot(0, 0, j % (w.history_chunks + 1))
        assert np.array_equal(a[0].view(np.uint32), b[0].view(np.uint32)) and np.array_equal(a[1], b[1])


# ----------------------------------------------------------------------------- ring bookkeeping and isolation

def test_ring_state_sequence():
    w = W.scaled(TINY, anchor_policy="none", total_frames=9)
    orc = make_oracle(w, O.BF16)
    H = w.history_chunks
    for i in range(w.n_chunks):
        for stage in reversed(range(w.n_stages)):
            q, k, v = (t.float().numpy() for t in W.qkv(w, 0, i, stage, 0, 1))
            assert orc.chunk_forward(stage, 0, i, 1, i, q, k, v)[0] == O.OK
            assert orc.advance(stage) == O.OK
            s = orc.ring_state(stage)
            n = i + 1
            assert s["head"] == n % (H + 1) and s["count"] == min(n, H) and s["next_chunk"] == n
            want = [-1] * (H + 1)
            for j in range(max(0, i - H), i + 1):
                want[j % (H + 1)] = j
            assert s["slot_chunk"] == want
    # out-of-order chunk index is refused and changes nothing
    q, k, v = (t.float().numpy() for t in W.qkv(w, 0, 0, 0, 0, 1))
    assert orc.chunk_forward(0, 0, 3, 1, 3, q, k, v)[0] == O.ERR_STATE
    assert orc.ring_state(0)["next_chunk"] == w.n_chunks


def test_everything_outside_the_visible_set_is_ignored():
    """Poisoning the evicted slot, other stages' banks, other layers and unused anchor slots with NaN leaves
    outputs and visible cache contents bit-identical."""
    w = W.scaled(TINY, n_layers=2, total_frames=5, n_anchor_slots=3)
    ref = make_oracle(w, O.BF16)
    want = run_stream(w, ref, O.BF16, seed=8)
    orc = make_oracle(w, O.BF16)
    H = w.history_chunks
    # an anchor slot nobody reads, published then poisoned
    k, v = W.anchor_kv(w, 8, 99, 0)
    for l in range(w.n_layers):
        assert orc.anchor_publish(2, 77, l, k.float().numpy(), v.float().numpy()) == O.OK
        orc.poison(1, 0, l, 2)
    got = {}
    for ev in W.trace(w):
        if ev.kind == "anchor":
            for l in range(w.n_layers):
                k, v = W.anchor_kv(w, 8, ev.anchor_id, l)
                orc.anchor_publish(ev.slot, ev.frame_pos, l, k.float().numpy(), v.float().numpy())
            continue
        i = ev.chunk
        for stage in reversed(range(w.n_stages)):
            for l in range(w.n_layers):
                # poison what this call must not see: the slot it is about to overwrite (chunk i-H-1),
                # the same slot indices in the other stage, and the other layer of this stage
                orc.poison(0, stage, l, i % (H + 1))
                other_stage = 1 - stage
                saved = [orc.ring_slot(other_stage, ll, s) for ll in range(w.n_layers) for s in range(H + 1)]
                for ll in range(w.n_layers):
                    for s in range(H + 1):
                        orc.poison(0, other_stage, ll, s)
                q, k, v = W.qkv(w, 8, i, stage, l, ev.n_frames)
                st, out = orc.chunk_forward(stage, l, i, ev.n_frames, ev.first_frame_pos, q.float().numpy(),
                                            k.float().numpy(), v.float().numpy(), ev.anchor_slots)
                assert st == O.OK
                got[(i, stage, l)] = out
                # restore the other stage's bank (it is needed by that stage's own later calls)
                it = iter(saved)
                for ll in range(w.n_layers):
                    for s in range(H + 1):
                        ks, vs = next(it)
                        _restore(orc, other_stage, ll, s, ks, vs)
            assert orc.advance(stage) == O.OK
    for key in want:
        assert np.array_equal(want[key].view(np.uint32), got[key].view(np.uint32)), key
    for stage in range(w.n_stages):
        for l in range(w.n_layers):
            for s in range(H + 1):
                a, b = ref.ring_slot(stage, l, s), orc.ring_slot(stage, l, s)
                if ref.ring_state(stage, l)["slot_chunk"][s] >= w.n_chunks - 1 - H:
                    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def _restore(orc, stage, layer, slot, k, v):
    import ctypes as C
    kp, vp, n = C.POINTER(C.c_float)(), C.POINTER(C.c_float)(), C.c_int32()
    O.lib().ffo_slot_data(orc._h, 0, stage, layer, slot, C.byref(kp), C.byref(vp), C.byref(n))
    if n.value:
        C.memmove(kp, k.ctypes.data, k.nbytes)
        C.memmove(vp, v.ctypes.data, v.nbytes)


def test_sampled_rows_equal_full_rows():
    w = W.scaled(TINY, anchor_policy="none")
    a, b = make_oracle(w, O.BF16), make_oracle(w, O.BF16)
    q, k, v = (t.float().numpy() for t in W.qkv(w, 0, 0, 0, 0, 1))
    _, full = a.chunk_forward(0, 0, 0, 1, 0, q, k, v)
    rows = [0, 5, 63]
    _, part = b.chunk_forward(0, 0, 0, 1, 0, q, k, v, rows=rows)
    assert np.array_equal(full[rows], part)


def test_published_cache_is_bf16_rotation_of_k_and_raw_v():
    w = W.scaled(TINY, anchor_policy="none")
    orc = make_oracle(w, O.BF16)
    q, k, v = W.qkv(w, 0, 0, 1, 0, 1)
    orc.chunk_forward(1, 0, 0, 1, 4, q.float().numpy(), k.float().numpy(), v.float().numpy())
    ck, cv = orc.ring_slot(1, 0, 0)
    assert np.array_equal(cv, v.float().numpy())
    pos = P.token_positions(1, 4, w.grid_h, w.grid_w)[:, None, :]
    want = P.rope_complex(k.float().numpy(), pos)
    # rounded to bf16: error at most half a bf16 ulp (2^-9 relative) plus the float rotation error
    assert np.all(np.abs(ck - want) <= np.abs(want) * 2.0 ** -8 + 1e-6)
    assert np.array_equal(torch.from_numpy(ck).to(torch.bfloat16).float().numpy(), ck)


# ----------------------------------------------------------------------------- q/k normalisation ahead of the rotation

@pytest.mark.parametrize("d,group", [(128, 8), (128, 4), (64, 8), (64, 4)])
def test_rms_norm_unit_rms_direction_and_float64_value(d, group):
    rng = np.random.default_rng(d + group)
    for scale in (1e-3, 1.0, 37.0):
        x = (rng.standard_normal(d) * scale).astype(np.float32)
        y = O.rms_norm_vec(x, eps=0.0, group=group)
        assert abs(math.sqrt(float(np.mean(y.astype(np.float64) ** 2))) - 1.0) < 1e-6
        want = x.astype(np.float64) / math.sqrt(float(np.mean(x.astype(np.float64) ** 2)))
        assert np.max(np.abs(y - want)) <= 4e-7 * np.max(np.abs(want))
        # same direction: the ratio y/x is one constant
        r = y[np.abs(x) > 1e-3 * scale] / x[np.abs(x) > 1e-3 * scale]
        assert np.ptp(r) <= 4e-7 * abs(r[0])


def test_rms_norm_power_of_two_scale_invariance_is_exact_and_eps_matters():
    rng = np.random.default_rng(5)
    x = rng.standard_normal(128).astype(np.float32)
    base = O.rms_norm_vec(x, eps=0.0)
    for c in (0.25, 8.0, 1024.0):           # scaling by 2^k commutes with every rounding
        assert np.array_equal(O.rms_norm_vec(x * np.float32(c), eps=0.0), base)
    # eps enters under the root: a vector of tiny entries is NOT blown up to unit rms
    tiny = np.full(128, 1e-4, dtype=np.float32)
    y = O.rms_norm_vec(tiny, eps=1e-6)
    assert np.allclose(y, 1e-4 / math.sqrt(1e-8 + 1e-6), rtol=1e-6)
    # and a zero vector stays zero (no 0/0)
    assert np.array_equal(O.rms_norm_vec(np.zeros(64, np.float32), eps=1e-6), np.zeros(64, np.float32))


def test_rms_norm_gain_is_per_channel_and_applied_last():
    rng = np.random.default_rng(6)
    x = rng.standard_normal(64).astype(np.float32)
    g = (rng.random(64) + 0.5).astype(np.float32)
    assert np.array_equal(O.rms_norm_vec(x, gain=g), O.rms_norm_vec(x) * g)
    e = np.zeros(64, np.float32)
    e[17] = 2.0
    assert np.array_equal(O.rms_norm_vec(x, gain=np.ones(64, np.float32) + e)[np.arange(64) != 17],
                          O.rms_norm_vec(x)[np.arange(64) != 17])


@pytest.mark.parametrize("dtype", [O.BF16, O.F32])
def test_cache_with_fused_norm_equals_cache_fed_normalised_rows(dtype):
    """Special case that reduces to the path without the option: normalising inside gives (up to the rounding of
    the intermediate) what the plain path gives on rows normalised beforehand in float64."""
    w = W.scaled(TINY, anchor_policy="none", total_frames=2)
    td = tdtype(dtype)
    a = make_oracle(w, dtype, qk_norm=True, qk_norm_eps=0.0)
    b = make_oracle(w, dtype)
    for i in range(2):
        q, k, v = W.qkv(w, 3, i, 1, 0, 1, td, pre_normalised=False)
        qn, kn = (x.double() / x.double().pow(2).mean(-1, keepdim=True).sqrt() for x in (q, k))
        st, oa = a.chunk_forward(1, 0, i, 1, i, q.float().numpy(), k.float().numpy(), v.float().numpy())
        assert st == O.OK
        st, ob = b.chunk_forward(1, 0, i, 1, i, qn.float().numpy(), kn.float().numpy(), v.float().numpy())
        assert st == O.OK
        ka, va = a.ring_slot(1, 0, i % (w.history_chunks + 1))
        kb, vb = b.ring_slot(1, 0, i % (w.history_chunks + 1))
        assert np.array_equal(va, vb)                      # V is never normalised
        ulp = 2.0 ** -7 if dtype == O.BF16 else 2.0 ** -21
        assert np.max(np.abs(ka - kb)) <= ulp * np.max(np.abs(kb))
        assert np.max(np.abs(oa - ob)) <= (3e-2 if dtype == O.BF16 else 1e-5)
        assert a.advance(1) == O.OK and b.advance(1) == O.OK


def test_fused_norm_gains_are_per_layer_and_separate_for_q_and_k():
    w = W.scaled(TINY, anchor_policy="none", n_layers=2)
    orc = make_oracle(w, O.F32, qk_norm=True)
    gq, gk = W.channel_gains(w, 0, 1)
    assert orc.set_qk_gain(1, gq.numpy(), gk.numpy()) == O.OK
    q, k, v = W.qkv(w, 0, 0, 0, 0, 1, torch.float32, pre_normalised=False)
    outs = []
    for layer in range(2):
        st, _ = orc.chunk_forward(0, layer, 0, 1, 0, q.numpy(), k.numpy(), v.numpy())
        assert st == O.OK
        outs.append(orc.ring_slot(0, layer, 0)[0])
    # layer 0 keeps unit gains; layer 1's keys are layer 0's keys with the k-gain applied before the rotation:
    # undo the rotation (rotate by the negated position) and compare channel by channel
    pos = P.token_positions(1, 0, w.grid_h, w.grid_w)
    t, h = 5, 1
    back0 = O.rope_vec(outs[0][t, h], -pos[t])
    back1 = O.rope_vec(outs[1][t, h], -pos[t])
    assert np.allclose(back1, back0 * gk.numpy(), rtol=2e-6, atol=1e-6)
    assert not np.allclose(back1, back0 * gq.numpy(), rtol=1e-3)


# ----------------------------------------------------------------------------- the update after the forward

def test_euler_step_follows_the_straight_flow_line_to_the_clean_latent():
    """With the exact velocity v = eps - x0, one step from sigma_k lands on x_{sigma_{k-1}}, and S steps from pure
    noise land on x0 (rectified-flow parameterisation; Alg. 1 "Step")."""
    rng = np.random.default_rng(11)
    x0 = rng.standard_normal(1000).astype(np.float32)
    eps = rng.standard_normal(1000).astype(np.float32)
    v = eps - x0
    sig = P.sigma_schedule(4, 5.0)
    x = P.flow_point(x0, eps, sig[4]).astype(np.float32)
    assert np.array_equal(x, eps)                           # sigma_S = 1: pure noise
    for k in range(4, 0, -1):
        x = O.euler_step(x, v, sig[k], sig[k - 1])
        assert np.max(np.abs(x - P.flow_point(x0, eps, sig[k - 1]))) < 2e-6
    assert np.max(np.abs(x - x0)) < 2e-6


def test_euler_step_sign_order_and_bf16_rounding():
    x = np.array([1.0, -2.0, 0.5], np.float32)
    v = np.array([2.0, 2.0, -4.0], np.float32)
    # sigma falls from 0.75 to 0.25: the latent moves AGAINST the velocity by half of it
    assert np.array_equal(O.euler_step(x, v, 0.75, 0.25), np.array([0.0, -3.0, 2.5], np.float32))
    assert np.array_equal(O.euler_step(x, v, 0.25, 0.25), x)
    r = O.euler_step(np.array([1.0], np.float32), np.array([1.0], np.float32), 2.0 ** -9, 0.0, round_bf16=True)
    assert r[0] == 1.0                                     # 1 - 2^-9 ties to even in bf16
    r = O.euler_step(np.array([1.0], np.float32), np.array([1.0], np.float32), 3 * 2.0 ** -9, 0.0, round_bf16=True)
    assert r[0] == np.float32(0.9921875)                   # halfway between 0x3F7E and 0x3F7F: the even one


def test_sigma_schedule_matches_the_printed_stage_indices():
    import json
    import os
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))["student_schedule"]
    sig = P.sigma_schedule(gold["n_stages"], gold["flow_shift"])
    assert sig[0] == 0.0 and sig[-1] == 1.0
    assert all(a < b for a, b in zip(sig, sig[1:]))
    # ordered from the highest noise level (stage S) down to stage 1
    for q, s in zip(gold["indices_high_to_low"], reversed(sig[1:])):
        assert abs(1000.0 * s - q) <= 1.0
