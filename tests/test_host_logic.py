"""CPU-only checks of the product's host side: the shared library loads and exports every symbol the header
declares, the bookkeeping-only cache follows the same ring/anchor sequence as the oracle, and the call counters
match the paper's forward-count model."""
import os
import re

import pytest

import ff_workloads as W
from oracle import ff_oracle as O
from oracle import paper_defs as PD

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2609_32540_b200 import build
    build.build()          # nvcc cross-compiles without a GPU
    from paper_2609_32540_b200 import binding
    binding.load()
    return binding


def test_library_exports_every_declared_symbol(B):
    header = open(os.path.join(ROOT, "include", "ff.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ff_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(B.SYMBOLS), declared ^ set(B.SYMBOLS)
    lib = B.load()
    for name in declared:
        assert hasattr(lib, name), name
    assert "sm_100a" in B.ff_version()


def test_arena_sizes_of_the_benchmark_configs(B):
    sizes = {}
    for name, w in W.CONFIGS.items():
        cfg = B.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h,
                            grid_w=w.grid_w, chunk_frames=w.chunk_frames, n_stages=w.n_stages,
                            history_chunks=w.history_chunks, n_anchor_slots=w.n_anchor_slots,
                            max_visible_anchors=w.visible_anchors, device=B.FF_DEVICE_NONE)
        sizes[name] = B.ff_cache_query_bytes(cfg)
    # rings: S*Ly*(H+1) slots of roundup128(B_R*T_f) rows of Hd*d bf16, K and V
    w = W.CONFIGS["wan1p3b_480p"]
    ring = 4 * 30 * 3 * 4736 * 12 * 128 * 2 * 2
    assert ring < sizes["wan1p3b_480p"] < ring * 1.1
    assert 100e9 < sizes["wan14b_720p_stream35s"] < 125e9      # fits one 180 GB GPU
    bad = B.make_config(n_layers=1, n_heads=1, head_dim=96, grid_h=2, grid_w=2, chunk_frames=1, n_stages=1,
                        history_chunks=1, n_anchor_slots=0, max_visible_anchors=0, device=B.FF_DEVICE_NONE)
    with pytest.raises(B.FFError) as e:
        B.ff_cache_query_bytes(bad)
    assert e.value.status == B.FF_ERR_UNSUPPORTED


def _dry_cache(B, w):
    cfg = B.make_config(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h,
                        grid_w=w.grid_w, chunk_frames=w.chunk_frames, n_stages=w.n_stages,
                        history_chunks=w.history_chunks, n_anchor_slots=w.n_anchor_slots,
                        max_visible_anchors=min(max(1, w.visible_anchors), w.n_anchor_slots),
                        device=B.FF_DEVICE_NONE)
    return B.Cache(cfg, None, 0)


def test_bookkeeping_follows_the_oracle_through_a_stream(B):
    """Ring head / count / next chunk / slot table after every advance, and anchor-slot table after every
    publish, against the oracle's (which is pinned to Eq. 2 by its own tests)."""
    import torch
    w = W.scaled(W.CONFIGS["tiny"], n_layers=2, total_frames=8, chunk_frames=3, grid_h=2, grid_w=2)
    c = _dry_cache(B, w)
    orc = O.Oracle(w.n_layers, w.n_heads, w.head_dim, w.grid_h, w.grid_w, w.chunk_frames, w.n_stages,
                   w.history_chunks, w.n_anchor_slots)
    p = 0x1000   # dummy aligned "device" pointers: nothing is enqueued in bookkeeping-only mode
    for ev in W.trace(w):
        if ev.kind == "anchor":
            for l in range(w.n_layers):
                k, v = W.anchor_kv(w, 0, ev.anchor_id, l)
                assert c.ff_anchor_publish(ev.slot, ev.frame_pos, l, p, p) == 0
                assert orc.anchor_publish(ev.slot, ev.frame_pos, l, k.float().numpy(), v.float().numpy()) == 0
            st = c.ff_cache_anchor_state(ev.slot)
            assert st["frame_pos"] == orc.anchor_frame_pos(ev.slot) == ev.frame_pos and all(st["layer_valid"])
            continue
        for stage in reversed(range(w.n_stages)):
            for l in range(w.n_layers):
                assert c.ff_chunk_forward_attn(stage, l, ev.chunk, ev.n_frames, ev.first_frame_pos, p, p, p,
                                               ev.anchor_slots, p) == 0
                q, k, v = W.qkv(w, 0, ev.chunk, stage, l, ev.n_frames)
                assert orc.chunk_forward(stage, l, ev.chunk, ev.n_frames, ev.first_frame_pos, q.float().numpy(),
                                         k.float().numpy(), v.float().numpy(), ev.anchor_slots, rows=[])[0] == 0
            assert c.ff_cache_advance(stage) == 0 and orc.advance(stage) == 0
            for l in range(w.n_layers):
                assert c.ff_cache_ring_state(stage, l) == orc.ring_state(stage, l)
    assert w.chunk_frames_of(w.n_chunks - 1) == 2        # the short last chunk is recorded with its token count
    assert c.ff_cache_ring_state(0, 0)["slot_tokens"][(w.n_chunks - 1) % 3] == 2 * w.tokens_per_frame
    cnt = c.ff_cache_counters()
    assert cnt["kernel_launches"] == 0                   # bookkeeping only


def test_call_counters_match_the_forward_count_model(B):
    """A whole L = 81 stream with one layer issues N_R*S layer-calls and N_R*S advances and not a single
    cache-update-only call; with the planner's N_P*(S+1) forwards that is W_FF = 123 of Eq. 3."""
    L, S = 81, 4
    w = W.Workload("count", 1, 1, 64, 2, 2, 3, S, 5, L, 0, 0, "none", 10)
    c = _dry_cache(B, w)
    p = 0x1000
    for i in range(w.n_chunks):
        io = [(p, p, p, p)]
        assert c.ff_sched_run_chunk(i, w.chunk_frames_of(i), 3 * i, [], io) == 0
    cnt = c.ff_cache_counters()
    fc = PD.forward_counts(L, S)
    assert cnt["layer_calls"] == fc["N_R"] * S == 108 and cnt["advances"] == fc["N_R"] * S
    assert fc["N_P"] * (S + 1) + cnt["layer_calls"] == fc["W_FF"] == 123
    s = c.ff_cache_ring_state(0)
    assert s["count"] == 5 and s["next_chunk"] == 27 and s["head"] == 27 % 6


def test_wavefront_order_is_accepted_and_wrong_orders_are_refused(B):
    w = W.Workload("wf", 2, 1, 64, 2, 2, 1, 4, 2, 6, 0, 0, "none", 1)
    p = 0x1000
    io = [(p, p, p, p)] * w.n_layers
    c = _dry_cache(B, w)
    for rnd in PD.wavefront_rounds(w.n_chunks, w.n_stages):
        for (i, k) in rnd:
            assert c.ff_sched_run_node(k - 1, i, 1, i, [], io) == 0
    for stage in range(w.n_stages):
        assert c.ff_cache_ring_state(stage)["next_chunk"] == w.n_chunks
    c2 = _dry_cache(B, w)
    assert c2.ff_sched_run_node(0, 1, 1, 1, [], io) == B.FF_ERR_STATE      # chunk 1 before chunk 0 at this stage
    assert c2.ff_chunk_forward_attn(0, 0, 0, 1, 0, p, p, p, [], p) == 0
    assert c2.ff_cache_advance(0) == B.FF_ERR_STATE                          # layer 1 has not run yet


def test_paper_index_helpers_match_the_paper_and_the_oracle(B):
    """ff_plan_* against the values the paper prints (worked example) and against the oracle's definitions, which
    are pinned to the paper on their own."""
    import json
    gold = json.load(open(os.path.join(ROOT, "tests", "golden", "paper_values.json")))["worked_example"]
    L, d, BR = gold["L"], gold["delta"], gold["B_R"]
    assert B.ff_plan_anchor_count(L, d) == gold["n_anchors"]
    assert [B.ff_plan_anchor_position(L, d, m) for m in range(gold["n_anchors"])] == gold["anchor_positions"]
    assert [B.ff_plan_anchor_position(L, d, m) for m in B.ff_plan_window(2, L, BR, d)] == \
        gold["chunk_at_positions_6_to_8_reads"]
    for (L, d, BR) in [(81, 10, 3), (21, 10, 3), (141, 10, 3), (261, 10, 3), (75, 10, 3), (5, 10, 3), (37, 4, 2)]:
        pos = PD.anchor_positions(L, d)
        assert B.ff_plan_anchor_count(L, d) == len(pos)
        assert [B.ff_plan_anchor_position(L, d, m) for m in range(len(pos))] == pos
        assert B.ff_plan_anchor_position(L, d, len(pos)) == -1
        for i in range(PD.n_chunks(L, BR)):
            got = [B.ff_plan_anchor_position(L, d, m) for m in B.ff_plan_window(i, L, BR, d)]
            assert got == PD.gamma_paper(i, L, BR, d), (L, d, BR, i)


def test_paper_budget_workload_uses_the_papers_window():
    w = W.PAPER_480P
    assert (w.history_chunks, w.visible_anchors, w.anchor_period_frames, w.total_frames) == (5, 3, 10, 81)
    assert PD.history_lengths(21, 3, 3) == (W.PAPER_480P_PLANNER.history_chunks, w.history_chunks)
    for i in range(w.n_chunks):
        got = [W.anchor_frame_pos(w, m) for m in W.visible_anchor_ids(w, i)]
        assert got == PD.gamma_paper(i, w.total_frames, w.chunk_frames, w.anchor_period_frames), i
    assert w.steady_n_kv() == 21 * w.tokens_per_frame == 32760      # W_ctx = 21 latent positions
    # the planner reads up to 18 earlier anchor latents plus its own block of 3
    assert W.PAPER_480P_PLANNER.steady_n_kv() == 21 * w.tokens_per_frame


def test_sigma_helper_matches_the_closed_form_and_rejects_bad_arguments(B):
    assert [B.ff_plan_sigma(k, 4, 5.0) for k in range(5)] == PD.sigma_schedule(4, 5.0)
    assert B.ff_plan_sigma(4, 4, 5.0) == 1.0 and B.ff_plan_sigma(0, 4, 5.0) == 0.0
    assert B.ff_plan_sigma(2, 4, 1.0) == 0.5           # shift 1: the uniform levels themselves
    for k, S, shift in [(-1, 4, 5.0), (5, 4, 5.0), (1, 0, 5.0), (1, 4, 0.0)]:
        with pytest.raises(B.FFError) as e:
            B.ff_plan_sigma(k, S, shift)
        assert e.value.status == B.FF_ERR_INVALID_ARG


def test_qk_norm_option_validation_and_arena_growth(B):
    w = W.CONFIGS["tiny"]
    kw = dict(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
              chunk_frames=w.chunk_frames, n_stages=w.n_stages, history_chunks=w.history_chunks,
              n_anchor_slots=w.n_anchor_slots, max_visible_anchors=1, device=B.FF_DEVICE_NONE)
    off = B.ff_cache_query_bytes(B.make_config(**kw))
    on = B.ff_cache_query_bytes(B.make_config(**kw, qk_norm=1, qk_norm_eps=1e-6))
    assert 0 < on - off <= 1024 + w.n_layers * 2 * w.head_dim * 4   # only the gain table is added
    with pytest.raises(B.FFError) as e:
        B.ff_cache_query_bytes(B.make_config(**kw, qk_norm=1, qk_norm_eps=-1.0))
    assert e.value.status == B.FF_ERR_INVALID_ARG
    c = B.Cache(B.make_config(**kw, qk_norm=1), None, 0)
    assert c.ff_cache_set_qk_gain(0, [1.0] * w.head_dim, [2.0] * w.head_dim) == B.FF_OK
    assert c.ff_cache_set_qk_gain(w.n_layers, [1.0] * w.head_dim, None) == B.FF_ERR_INVALID_ARG
    c.close()
    c = B.Cache(B.make_config(**kw), None, 0)
    assert c.ff_cache_set_qk_gain(0, [1.0] * w.head_dim, None) == B.FF_ERR_STATE
    c.close()


def _check_schedule(B, n_heads, n_q, n_kv, n_ctas_max=148, unit_pairs=1):
    """unit_pairs = 2: the kernel on CTA pairs; a unit is two consecutive pairs of query tiles, a slot a CTA pair."""
    hdr, pieces = B.ff_debug_schedule(n_heads, n_q, n_kv, n_ctas_max, unit_pairs)
    tiles = [-(-k // 128) for k in n_kv]
    n_qt = [-(-q // 128) for q in n_q]
    n_qp = [-(-((t + 1) // 2) // unit_pairs) for t in n_qt]     # units per head
    cover = {}
    per_cta = {}
    slots_seen = set()
    for cta, item, h, pr, j0, j1, slot, two in pieces:
        assert 0 <= item < len(n_q) and 0 <= h < n_heads and 0 <= pr < n_qp[item]
        assert 0 <= j0 < j1 <= tiles[item]
        if unit_pairs == 1:
            assert bool(two) == (2 * pr + 1 < n_qt[item])
        whole = j0 == 0 and j1 == tiles[item]
        if whole:
            assert slot == -1
        else:
            assert slot in (2 * cta, 2 * cta + 1) and slot not in slots_seen   # a scratch slot is written once
            slots_seen.add(slot)
        for j in range(j0, j1):
            key = (item, h, pr, j)
            assert key not in cover, "key tile visited twice"
            cover[key] = cta
        per_cta[cta] = per_cta.get(cta, 0) + (j1 - j0)
    want = sum(n_heads * n_qp[i] * tiles[i] for i in range(len(n_q)))
    assert len(cover) == want, "some (pair, key tile) never visited"
    assert hdr["n_ctas"] <= n_ctas_max and max(per_cta) < hdr["n_ctas"]
    # balance: CTAs differ by at most the spread of whole pairs plus one share rounding
    if len(set(tiles)) == 1:
        assert max(per_cta.values()) - min(per_cta.values()) <= hdr["iters_per_cta"]
    # pieces of a cut pair, and the scratch slot the merge step derives for each: 2c when CTA c's share of the
    # flattened remainder list begins inside the pair's range of that list, else 2c + 1
    order = [(i, h, pr) for i in range(len(n_q)) for h in range(n_heads) for pr in range(n_qp[i])]
    g0 = hdr["n_full"] * hdr["n_ctas"]
    start, pos = {}, 0
    for key in order[g0:]:
        start[key] = pos
        pos += tiles[key[0]]
    cut = {}
    for cta, item, h, pr, j0, j1, slot, two in pieces:
        if slot >= 0:
            cut.setdefault((item, h, pr), []).append((j0, j1, cta, slot))
    assert bool(cut) == (hdr["merge_pairs"] > 0)
    if cut:
        assert hdr["merge_pairs"] == len(order) - g0
    for key, ps in cut.items():
        ps.sort()
        s_g, e_g = start[key], start[key] + tiles[key[0]]
        assert ps[0][0] == 0 and ps[-1][1] == tiles[key[0]] and all(a[1] == b[0] for a, b in zip(ps, ps[1:]))
        assert [p[2] for p in ps] == list(range(s_g // hdr["iters_per_cta"], (e_g - 1) // hdr["iters_per_cta"] + 1))
        for j0, j1, cta, slot in ps:
            c0 = cta * hdr["iters_per_cta"]
            assert slot == 2 * cta + (0 if s_g <= c0 < e_g else 1)
    return hdr, pieces


@pytest.mark.parametrize("n_heads,n_q,n_kv", [
    (12, [4680], [15600]),                              # the 480p headline call
    (12, [4680] * 4, [15600] * 4),                      # a full wavefront round of it
    (12, [4680] * 4, [4680, 10920, 15600, 15600]),      # ramp-up: stages see different history lengths
    (40, [10800] * 4, [36000] * 4),                     # 14B 720p round
    (2, [64], [128 + 64]), (2, [64, 64], [64, 192]),    # tiny
    (3, [414, 207], [1449, 621]),                       # ragged, short last chunk in one stage
    (1, [129], [1]), (5, [1000] * 8, [3000] * 8),
    # more layer-calls than travel as launch arguments (descriptor table): a clip's chunks in one launch, with the
    # warm-up chunks seeing fewer keys and a short last chunk
    (12, [4680] * 27, [min(i + 1, 6) * 4680 + 3 * 1560 for i in range(27)]),
    (2, [64] * 9, [64 * min(i + 1, 3) for i in range(9)]),
    (3, [300] * 40 + [100], [300 * min(i + 1, 4) + 77 for i in range(40)] + [1377]),
])
def test_attention_work_distribution_covers_everything_once(B, n_heads, n_q, n_kv):
    for n_ctas in (148, 7, 1):
        _check_schedule(B, n_heads, n_q, n_kv, n_ctas)
    for n_pairs_of_ctas in (74, 5, 1):
        _check_schedule(B, n_heads, n_q, n_kv, n_pairs_of_ctas, unit_pairs=2)


def test_same_stage_batches_follow_the_slot_rule(B):
    """Consecutive chunks of one stage may share a batch when the bank has H + n slots (bookkeeping-only cache)."""
    w = W.scaled(W.CONFIGS["tiny"], anchor_policy="none", n_anchor_slots=0)
    H = w.history_chunks
    kw = dict(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
              chunk_frames=w.chunk_frames, n_stages=w.n_stages, history_chunks=H, n_anchor_slots=0,
              max_visible_anchors=0, device=B.FF_DEVICE_NONE)
    for bad in (dict(ring_slots=H), dict(ring_slots=5000), dict(max_batch=B.FF_MAX_BATCH + 1), dict(max_batch=-1)):
        with pytest.raises(B.FFError) as e:
            B.ff_cache_query_bytes(B.make_config(**kw, **bad))
        assert e.value.status == B.FF_ERR_INVALID_ARG
    small = B.ff_cache_query_bytes(B.make_config(**kw))
    big = B.ff_cache_query_bytes(B.make_config(**kw, ring_slots=H + 3, max_batch=4))
    assert big > small
    c = B.Cache(B.make_config(**kw, ring_slots=H + 3, max_batch=4), None, 0)

    def item(stage, chunk):
        return dict(stage=stage, chunk_index=chunk, n_frames=1, first_frame_pos=chunk, q=16, k=16, v=16, out=16)

    assert c.ff_batch_forward_attn(0, [item(1, 0), item(1, 1), item(1, 2), item(1, 3)]) == B.FF_ERR_UNSUPPORTED  # H+4 slots
    assert c.ff_batch_forward_attn(0, [item(1, 1), item(1, 0)]) == B.FF_ERR_STATE        # out of order
    assert c.ff_batch_forward_attn(0, [item(1, 0), item(1, 2)]) == B.FF_ERR_STATE        # gap
    assert c.ff_cache_counters()["layer_calls"] == 0
    # three chunks of stage 1 together with one chunk of stage 0
    assert c.ff_batch_forward_attn(0, [item(1, 0), item(0, 0), item(1, 1), item(1, 2)]) == B.FF_OK
    st = c.ff_cache_ring_state(1, 0)
    assert len(st["slot_chunk"]) == H + 3 and st["slot_chunk"][:3] == [0, 1, 2] and st["next_chunk"] == 0
    for n in range(3):
        assert c.ff_cache_advance(1) == B.FF_OK
    assert c.ff_cache_advance(1) == B.FF_ERR_STATE                                        # chunk 3 has not run
    st = c.ff_cache_ring_state(1, 0)
    assert st["next_chunk"] == 3 and st["count"] == H and st["head"] == 3 % (H + 3)
    # next group: chunks 3..5 wrap around the H + 3 slots; chunk 5 lands on slot 0 (chunk 0 is out of every window)
    assert c.ff_batch_forward_attn(0, [item(1, 3), item(1, 4), item(1, 5)]) == B.FF_OK
    assert c.ff_cache_ring_state(1, 0)["slot_chunk"][0] == 5
    c.close()


def test_a_refused_launch_leaves_the_tables_and_counters_untouched(B):
    """Host-injected launch failure (no GPU involved): whichever launch site of a call fails, the call returns
    FF_ERR_CUDA and the ring table, the anchor table and the counters are what they were; the same call then
    succeeds."""
    w = W.scaled(W.CONFIGS["tiny"], n_stages=2)
    c = _dry_cache(B, w)

    def snapshot():
        return ([c.ff_cache_ring_state(s, 0) for s in range(w.n_stages)], c.ff_cache_anchor_state(0), c.ff_cache_counters())

    before = snapshot()
    assert c.ff_debug_fail_launch(1) == B.FF_OK
    assert c.ff_anchor_publish(0, 3, 0, 16, 16) == B.FF_ERR_CUDA
    assert B.ff_last_cuda_error() != 0 and snapshot() == before
    assert c.ff_anchor_publish(0, 3, 0, 16, 16) == B.FF_OK
    before = snapshot()
    # a single call has two launch sites (publish, attention); a batch of two stages has the same two
    for nth in (1, 2):
        assert c.ff_debug_fail_launch(nth) == B.FF_OK
        assert c.ff_chunk_forward_attn(1, 0, 0, 1, 0, 16, 16, 16, [0], 16) == B.FF_ERR_CUDA
        assert snapshot() == before
        assert c.ff_cache_advance(1) == B.FF_ERR_STATE           # the chunk was never recorded as published
    items = [dict(stage=s, chunk_index=0, n_frames=1, first_frame_pos=0, q=16, k=16, v=16, out=16, anchor_slots=[0])
             for s in (1, 0)]
    assert c.ff_debug_fail_launch(2) == B.FF_OK
    assert c.ff_batch_forward_attn(0, items) == B.FF_ERR_CUDA and snapshot() == before
    assert c.ff_batch_forward_attn(0, items) == B.FF_OK
    after = snapshot()
    assert after[2]["layer_calls"] == before[2]["layer_calls"] + 2
    assert [st["slot_chunk"][0] for st in after[0]] == [0, 0]
    assert c.ff_cache_advance(1) == B.FF_OK and c.ff_cache_advance(0) == B.FF_OK
    assert c.ff_debug_fail_launch(-1) == B.FF_ERR_INVALID_ARG
    c.close()


def test_whole_clip_of_a_stage_in_one_batch(B):
    """All 27 chunks of the 81-latent clip as ONE batched call per layer (bookkeeping-only cache): needs H + 27 bank
    slots and 27 query regions; the later chunks see the earlier ones' token counts, the last chunk may be short."""
    w = W.scaled(W.PAPER_480P, n_layers=2, n_stages=1, grid_h=2, grid_w=4, total_frames=80)   # 26 chunks of 3 + one of 2
    N, H = w.n_chunks, w.history_chunks
    assert N == 27
    kw = dict(n_layers=w.n_layers, n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
              chunk_frames=w.chunk_frames, n_stages=1, history_chunks=H, n_anchor_slots=0, max_visible_anchors=0,
              device=B.FF_DEVICE_NONE)
    c = B.Cache(B.make_config(**kw, ring_slots=H + N, max_batch=N), None, 0)
    items = [dict(stage=0, chunk_index=i, n_frames=w.chunk_frames_of(i), first_frame_pos=3 * i, q=16, k=16, v=16, out=16)
             for i in range(N)]
    for l in range(w.n_layers):
        assert c.ff_batch_forward_attn(l, items) == B.FF_OK
    st = c.ff_cache_ring_state(0, 1)
    assert st["slot_chunk"][:N] == list(range(N)) and st["slot_tokens"][N - 1] == 2 * w.tokens_per_frame
    for i in range(N):
        assert c.ff_cache_advance(0) == B.FF_OK
    assert c.ff_cache_counters()["layer_calls"] == 2 * N
    c.close()
    small = B.Cache(B.make_config(**kw, ring_slots=H + N, max_batch=8), None, 0)
    assert small.ff_batch_forward_attn(0, items) == B.FF_ERR_UNSUPPORTED      # more calls than query regions
    small.close()


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    """There is no fallback: without the built shared library the binding raises instead of computing elsewhere."""
    from paper_2609_32540_b200 import binding, build
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(build, "LIB_PATH", str(tmp_path / "libff_chunk_attn.so"))
    with pytest.raises(ImportError):
        binding.load()
    with pytest.raises(ImportError):
        binding.ff_plan_sigma(1, 4, 5.0)
