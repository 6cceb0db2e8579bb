"""ctypes binding of the C ABI declared in include/ff.h: argument marshalling only.

Every step of the path (rotary embedding, cache publish, attention, ring bookkeeping, the stage scheduler) runs
inside the shared library.  PyTorch appears only as the owner of device memory and streams: callers pass
`tensor.data_ptr()` and `torch.cuda.current_stream().cuda_stream`.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

FF_OK, FF_ERR_INVALID_ARG, FF_ERR_STATE, FF_ERR_OOM, FF_ERR_UNSUPPORTED, FF_ERR_CUDA, FF_ERR_TIMEOUT = range(7)
FF_BF16, FF_F32 = 0, 1
FF_ATTN_AUTO, FF_ATTN_TCGEN05, FF_ATTN_SIMT, FF_ATTN_TCGEN05_PAIR = 0, 1, 2, 3
FF_DEVICE_NONE = -1

_STATUS_NAMES = ["FF_OK", "FF_ERR_INVALID_ARG", "FF_ERR_STATE", "FF_ERR_OOM", "FF_ERR_UNSUPPORTED", "FF_ERR_CUDA",
                 "FF_ERR_TIMEOUT"]

# every symbol include/ff.h declares
SYMBOLS = [
    "ff_cache_query_bytes", "ff_cache_create", "ff_cache_destroy", "ff_cache_reset", "ff_anchor_publish",
    "ff_chunk_forward_attn", "ff_cache_advance", "ff_chunk_forward_attn_host", "ff_sched_run_chunk",
    "ff_sched_run_chunk_host", "ff_sched_run_node", "ff_plan_anchor_count", "ff_plan_anchor_position",
    "ff_plan_window", "ff_cache_profile_begin", "ff_cache_profile_end",
    "ff_cache_ring_state", "ff_cache_anchor_state", "ff_cache_slot_ptr", "ff_cache_status",
    "ff_cache_counters", "ff_cache_kernel_choice", "ff_debug_wait_probe", "ff_debug_fail_launch", "ff_debug_set_trace", "ff_chunk_attn_static", "ff_cache_set_qk_gain",
    "ff_euler_step", "ff_plan_sigma", "ff_batch_forward_attn", "ff_sched_run_round", "ff_debug_schedule", "ff_last_cuda_error", "ff_version",
]


class FFError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        name = _STATUS_NAMES[status] if 0 <= status < len(_STATUS_NAMES) else str(status)
        super().__init__(f"{what}: {name}")


class ff_cache_config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("grid_h", C.c_int32), ("grid_w", C.c_int32), ("chunk_frames", C.c_int32),
        ("n_stages", C.c_int32), ("history_chunks", C.c_int32), ("n_anchor_slots", C.c_int32),
        ("max_visible_anchors", C.c_int32), ("dtype", C.c_int32), ("attn_impl", C.c_int32),
        ("max_frame_pos", C.c_int32), ("rope_pairs", C.c_int32 * 3), ("rope_theta", C.c_float),
        ("device", C.c_int32), ("frame_pos_stride", C.c_int32), ("allow_republish", C.c_int32),
        ("ring_slots", C.c_int32), ("max_batch", C.c_int32),
        ("qk_norm", C.c_int32), ("qk_norm_eps", C.c_float),
    ]


class ff_layer_io(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p), ("out", C.c_void_p)]


class ff_batch_item(C.Structure):
    _fields_ = [("stage", C.c_int32), ("chunk_index", C.c_int32), ("n_frames", C.c_int32),
                ("first_frame_pos", C.c_int32), ("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p),
                ("out", C.c_void_p), ("anchor_slots", C.POINTER(C.c_int32)), ("n_anchors", C.c_int32)]


class ff_round_node(C.Structure):
    _fields_ = [("stage", C.c_int32), ("chunk_index", C.c_int32), ("n_frames", C.c_int32),
                ("first_frame_pos", C.c_int32), ("anchor_slots", C.POINTER(C.c_int32)), ("n_anchors", C.c_int32),
                ("io", C.POINTER(ff_layer_io))]


FF_MAX_BATCH = 128
_lib = None


def load():
    """Loads the in-tree shared library; fails loudly if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2609_32540_b200.build` (needs nvcc) first")
    L = C.CDLL(path)
    i32, vp, i32p, i64p = C.c_int32, C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int64)
    cfgp = C.POINTER(ff_cache_config)
    L.ff_cache_query_bytes.argtypes = [cfgp, C.POINTER(C.c_size_t)]
    L.ff_cache_create.argtypes = [cfgp, vp, C.c_size_t, C.POINTER(vp)]
    L.ff_cache_destroy.argtypes = [vp]
    L.ff_cache_reset.argtypes = [vp]
    L.ff_anchor_publish.argtypes = [vp, i32, i32, i32, vp, vp, vp]
    L.ff_chunk_forward_attn.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, i32p, i32, vp, vp]
    L.ff_chunk_forward_attn_host.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, i32p, i32, vp, vp]
    L.ff_cache_advance.argtypes = [vp, i32]
    L.ff_sched_run_chunk.argtypes = [vp, i32, i32, i32, i32p, i32, C.POINTER(ff_layer_io), i32, vp]
    L.ff_sched_run_chunk_host.argtypes = [vp, i32, i32, i32, i32p, i32, C.POINTER(ff_layer_io), i32, vp]
    L.ff_cache_profile_begin.argtypes = [vp, i32]
    L.ff_cache_profile_end.argtypes = [vp, vp, C.POINTER(C.c_double), i64p, C.POINTER(C.c_double), i64p]
    L.ff_plan_anchor_count.argtypes = [i32, i32]
    L.ff_plan_anchor_position.argtypes = [i32, i32, i32]
    L.ff_plan_window.argtypes = [i32, i32, i32, i32, i32p]
    L.ff_sched_run_node.argtypes = [vp, i32, i32, i32, i32, i32p, i32, C.POINTER(ff_layer_io), vp]
    L.ff_cache_ring_state.argtypes = [vp, i32, i32, i32p, i32p, i32p, i32p, i32p]
    L.ff_cache_anchor_state.argtypes = [vp, i32, i32p, C.POINTER(C.c_uint8)]
    L.ff_cache_slot_ptr.argtypes = [vp, i32, i32, i32, i32, C.POINTER(vp), C.POINTER(vp), i64p, i32p]
    L.ff_cache_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    L.ff_cache_counters.argtypes = [vp, i64p, i64p, i64p, i64p]
    L.ff_cache_kernel_choice.argtypes = [vp, i64p, i64p]
    L.ff_debug_wait_probe.argtypes = [vp, C.c_uint64, vp]
    L.ff_debug_fail_launch.argtypes = [vp, i32]
    L.ff_debug_set_trace.argtypes = [vp, vp, i32]
    L.ff_chunk_attn_static.argtypes = [i32, i32, i32, i32, i32, i32, C.c_float, i32, vp, vp, vp, vp, vp]
    L.ff_cache_set_qk_gain.argtypes = [vp, i32, C.POINTER(C.c_float), C.POINTER(C.c_float), vp]
    L.ff_euler_step.argtypes = [vp, vp, C.c_float, C.c_float, C.c_int64, i32, i32, vp, vp]
    L.ff_plan_sigma.argtypes = [i32, i32, C.c_double, C.POINTER(C.c_double)]
    L.ff_batch_forward_attn.argtypes = [vp, i32, C.POINTER(ff_batch_item), i32, vp]
    L.ff_sched_run_round.argtypes = [vp, C.POINTER(ff_round_node), i32, vp]
    L.ff_debug_schedule.argtypes = [i32, i32, i32p, i32p, i32, i32, i32p, i32, i32p]
    L.ff_last_cuda_error.restype = i32
    L.ff_version.restype = C.c_char_p
    for name in SYMBOLS:
        fn = getattr(L, name)
        if name not in ("ff_last_cuda_error", "ff_version"):
            fn.restype = i32
    _lib = L
    return L


def make_config(*, n_layers, n_heads, head_dim, grid_h, grid_w, chunk_frames, n_stages, history_chunks,
                n_anchor_slots, max_visible_anchors, dtype=FF_BF16, attn_impl=FF_ATTN_AUTO, max_frame_pos=1024,
                rope_pairs=(0, 0, 0), rope_theta=10000.0, device=0, frame_pos_stride=1,
                allow_republish=0, qk_norm=0, qk_norm_eps=1e-6, ring_slots=0, max_batch=0) -> ff_cache_config:
    cfg = ff_cache_config()
    cfg.n_layers, cfg.n_heads, cfg.head_dim = n_layers, n_heads, head_dim
    cfg.grid_h, cfg.grid_w, cfg.chunk_frames = grid_h, grid_w, chunk_frames
    cfg.n_stages, cfg.history_chunks = n_stages, history_chunks
    cfg.n_anchor_slots, cfg.max_visible_anchors = n_anchor_slots, max_visible_anchors
    cfg.dtype, cfg.attn_impl, cfg.max_frame_pos = dtype, attn_impl, max_frame_pos
    cfg.rope_pairs = (C.c_int32 * 3)(*rope_pairs)
    cfg.rope_theta, cfg.device = rope_theta, device
    cfg.frame_pos_stride, cfg.allow_republish = frame_pos_stride, allow_republish
    cfg.qk_norm, cfg.qk_norm_eps = qk_norm, qk_norm_eps
    cfg.ring_slots, cfg.max_batch = ring_slots, max_batch
    return cfg


def _check(st: int, what: str):
    if st != FF_OK:
        raise FFError(st, what)


def _slots(anchor_slots):
    n = len(anchor_slots)
    return ((C.c_int32 * n)(*anchor_slots) if n else None), n


def ff_cache_query_bytes(cfg: ff_cache_config) -> int:
    n = C.c_size_t()
    _check(load().ff_cache_query_bytes(C.byref(cfg), C.byref(n)), "ff_cache_query_bytes")
    return n.value


class Cache:
    """Handle of one ff_cache.  `arena_ptr` is a device address the caller keeps alive (e.g. a torch uint8 tensor)."""

    def __init__(self, cfg: ff_cache_config, arena_ptr: int | None, arena_bytes: int):
        self.cfg = cfg
        self._h = C.c_void_p()
        _check(load().ff_cache_create(C.byref(cfg), C.c_void_p(arena_ptr or 0), arena_bytes, C.byref(self._h)),
               "ff_cache_create")

    def close(self):
        if self._h:
            load().ff_cache_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- the four calls of the path, plus host-buffer and scheduler entry points (raw status returned) ---
    def ff_cache_reset(self) -> int:
        return load().ff_cache_reset(self._h)

    def ff_cache_set_qk_gain(self, layer, gain_q=None, gain_k=None, stream=0) -> int:
        """gain_q / gain_k: sequences of head_dim floats (or None to leave that side as it is)."""
        def arr(g):
            return None if g is None else (C.c_float * len(g))(*[float(x) for x in g])
        return load().ff_cache_set_qk_gain(self._h, layer, arr(gain_q), arr(gain_k), stream)

    def ff_anchor_publish(self, slot, frame_pos, layer, k_ptr, v_ptr, stream=0) -> int:
        return load().ff_anchor_publish(self._h, slot, frame_pos, layer, k_ptr, v_ptr, stream)

    def ff_chunk_forward_attn(self, stage, layer, chunk_index, n_frames, first_frame_pos, q_ptr, k_ptr, v_ptr,
                              anchor_slots, out_ptr, stream=0) -> int:
        arr, n = _slots(anchor_slots)
        return load().ff_chunk_forward_attn(self._h, stage, layer, chunk_index, n_frames, first_frame_pos, q_ptr,
                                            k_ptr, v_ptr, arr, n, out_ptr, stream)

    def ff_chunk_forward_attn_host(self, stage, layer, chunk_index, n_frames, first_frame_pos, q_ptr, k_ptr, v_ptr,
                                   anchor_slots, out_ptr, stream=0) -> int:
        arr, n = _slots(anchor_slots)
        return load().ff_chunk_forward_attn_host(self._h, stage, layer, chunk_index, n_frames, first_frame_pos,
                                                 q_ptr, k_ptr, v_ptr, arr, n, out_ptr, stream)

    def ff_cache_advance(self, stage) -> int:
        return load().ff_cache_advance(self._h, stage)

    def ff_sched_run_chunk(self, chunk_index, n_frames, first_frame_pos, anchor_slots, io, stream=0) -> int:
        """io: list of (q_ptr, k_ptr, v_ptr, out_ptr) or a prebuilt ff_layer_io array."""
        arr, n = _slots(anchor_slots)
        io_arr = io if isinstance(io, C.Array) else make_io(io)
        return load().ff_sched_run_chunk(self._h, chunk_index, n_frames, first_frame_pos, arr, n, io_arr,
                                         len(io_arr), stream)

    def ff_sched_run_chunk_host(self, chunk_index, n_frames, first_frame_pos, anchor_slots, io, stream=0) -> int:
        arr, n = _slots(anchor_slots)
        io_arr = io if isinstance(io, C.Array) else make_io(io)
        return load().ff_sched_run_chunk_host(self._h, chunk_index, n_frames, first_frame_pos, arr, n, io_arr,
                                              len(io_arr), stream)

    def ff_batch_forward_attn(self, layer, items, stream=0) -> int:
        """items: dicts with stage, chunk_index, n_frames, first_frame_pos, q, k, v, out (device pointers) and
        anchor_slots (a list)."""
        arr = (ff_batch_item * max(len(items), 1))()
        keep = []
        for i, it in enumerate(items):
            slots, n = _slots(list(it.get("anchor_slots", ())))
            keep.append(slots)
            arr[i] = ff_batch_item(it["stage"], it["chunk_index"], it["n_frames"], it["first_frame_pos"], it["q"],
                                   it["k"], it["v"], it["out"], slots, n)
        return load().ff_batch_forward_attn(self._h, layer, arr, len(items), stream)

    def ff_sched_run_round(self, nodes, stream=0) -> int:
        """nodes: dicts with stage, chunk_index, n_frames, first_frame_pos, anchor_slots (a list) and io (an
        ff_layer_io array of n_layers entries, see make_io)."""
        arr = (ff_round_node * max(len(nodes), 1))()
        keep = []
        for i, nd in enumerate(nodes):
            slots, n = _slots(list(nd.get("anchor_slots", ())))
            keep.append(slots)
            arr[i] = ff_round_node(nd["stage"], nd["chunk_index"], nd["n_frames"], nd["first_frame_pos"], slots, n,
                                   nd["io"])
        return load().ff_sched_run_round(self._h, arr, len(nodes), stream)

    def ff_cache_profile_begin(self, max_calls) -> int:
        return load().ff_cache_profile_begin(self._h, max_calls)

    def ff_cache_profile_end(self, stream=0) -> dict:
        pm, am, pn, an = C.c_double(), C.c_double(), C.c_int64(), C.c_int64()
        _check(load().ff_cache_profile_end(self._h, stream, C.byref(pm), C.byref(pn), C.byref(am), C.byref(an)),
               "ff_cache_profile_end")
        return dict(publish_ms=pm.value, publish_launches=pn.value, attn_ms=am.value, attn_launches=an.value)

    def ff_sched_run_node(self, stage, chunk_index, n_frames, first_frame_pos, anchor_slots, io, stream=0) -> int:
        arr, n = _slots(anchor_slots)
        io_arr = io if isinstance(io, C.Array) else make_io(io)
        assert len(io_arr) == self.cfg.n_layers
        return load().ff_sched_run_node(self._h, stage, chunk_index, n_frames, first_frame_pos, arr, n, io_arr,
                                        stream)

    # --- observers ---
    def ff_cache_ring_state(self, stage, layer=0) -> dict:
        n = self.cfg.ring_slots or self.cfg.history_chunks + 1
        head, count, nxt = C.c_int32(), C.c_int32(), C.c_int32()
        sc, stok = (C.c_int32 * n)(), (C.c_int32 * n)()
        _check(load().ff_cache_ring_state(self._h, stage, layer, C.byref(head), C.byref(count), C.byref(nxt), sc, stok),
               "ff_cache_ring_state")
        return dict(head=head.value, count=count.value, next_chunk=nxt.value, slot_chunk=list(sc),
                    slot_tokens=list(stok))

    def ff_cache_anchor_state(self, slot) -> dict:
        pos = C.c_int32()
        valid = (C.c_uint8 * self.cfg.n_layers)()
        _check(load().ff_cache_anchor_state(self._h, slot, C.byref(pos), valid), "ff_cache_anchor_state")
        return dict(frame_pos=pos.value, layer_valid=[bool(x) for x in valid])

    def ff_cache_slot_ptr(self, kind, stage, layer, slot) -> dict:
        k, v = C.c_void_p(), C.c_void_p()
        strides = (C.c_int64 * 3)()
        cap = C.c_int32()
        _check(load().ff_cache_slot_ptr(self._h, kind, stage, layer, slot, C.byref(k), C.byref(v), strides,
                                        C.byref(cap)), "ff_cache_slot_ptr")
        return dict(k=k.value, v=v.value, strides=tuple(strides), capacity_tokens=cap.value)

    def ff_cache_status(self, stream=0) -> tuple[int, int]:
        w = C.c_uint32()
        st = load().ff_cache_status(self._h, stream, C.byref(w))
        return st, w.value

    def ff_cache_counters(self) -> dict:
        a, b, c_, d = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64()
        _check(load().ff_cache_counters(self._h, C.byref(a), C.byref(b), C.byref(c_), C.byref(d)),
               "ff_cache_counters")
        return dict(layer_calls=a.value, advances=b.value, anchor_publishes=c_.value, kernel_launches=d.value)

    def ff_cache_kernel_choice(self) -> dict:
        a, b = C.c_int64(), C.c_int64()
        _check(load().ff_cache_kernel_choice(self._h, C.byref(a), C.byref(b)), "ff_cache_kernel_choice")
        return dict(one_cta=a.value, cta_pair=b.value)

    def ff_debug_set_trace(self, buf_ptr, cap) -> int:
        return load().ff_debug_set_trace(self._h, buf_ptr, cap)

    def ff_debug_fail_launch(self, nth) -> int:
        return load().ff_debug_fail_launch(self._h, nth)

    def ff_debug_wait_probe(self, limit_ns, stream=0) -> int:
        return load().ff_debug_wait_probe(self._h, limit_ns, stream)


def ff_plan_anchor_count(L, delta) -> int:
    return load().ff_plan_anchor_count(L, delta)


def ff_plan_anchor_position(L, delta, m) -> int:
    return load().ff_plan_anchor_position(L, delta, m)


def ff_plan_window(i, L, B_R, delta) -> list:
    out = (C.c_int32 * 3)()
    n = load().ff_plan_window(i, L, B_R, delta, out)
    return list(out[:n])


def make_io(entries):
    arr = (ff_layer_io * len(entries))()
    for i, (q, k, v, o) in enumerate(entries):
        arr[i].q, arr[i].k, arr[i].v, arr[i].out = q, k, v, o
    return arr


FF_STATIC_SCRATCH_BYTES = 8 * 1024 * 1024


def ff_chunk_attn_static(n_heads, head_dim, grid_h, grid_w, n_frames, first_frame_pos, rope_theta, dtype, q_ptr,
                         k_ptr, v_ptr, out_ptr, stream=0) -> int:
    """First-chunk layer-call that allocates nothing: its scratch is a fixed device array inside the library
    (FF_STATIC_SCRATCH_BYTES, shared by all calls on the device - keep them on one stream)."""
    return load().ff_chunk_attn_static(n_heads, head_dim, grid_h, grid_w, n_frames, first_frame_pos, rope_theta,
                                       dtype, q_ptr, k_ptr, v_ptr, out_ptr, stream)


def ff_euler_step(x_ptr, v_ptr, sigma_k, sigma_km1, n, dtype_x, dtype_v, out_ptr, stream=0) -> int:
    """out = x - (sigma_k - sigma_km1) * v over n elements (device pointers; out may equal x)."""
    return load().ff_euler_step(x_ptr, v_ptr, sigma_k, sigma_km1, n, dtype_x, dtype_v, out_ptr, stream)


def ff_plan_sigma(k, n_stages, shift=5.0) -> float:
    s = C.c_double()
    _check(load().ff_plan_sigma(k, n_stages, shift, C.byref(s)), "ff_plan_sigma")
    return s.value


def ff_debug_schedule(n_heads, n_q, n_kv, n_ctas_max=148, unit_pairs=1):
    """Host-only: (header dict, list of piece tuples) of a tensor-core kernel's work distribution (unit_pairs = 2:
    the kernel on CTA pairs, n_ctas_max then counts pairs)."""
    n = len(n_q)
    aq, ak = (C.c_int32 * n)(*n_q), (C.c_int32 * n)(*n_kv)
    hdr = (C.c_int32 * 4)()
    total = load().ff_debug_schedule(n_heads, n, aq, ak, n_ctas_max, unit_pairs, None, 0, hdr)
    if total < 0:
        raise FFError(FF_ERR_INVALID_ARG, "ff_debug_schedule")
    rec = (C.c_int32 * (8 * max(total, 1)))()
    load().ff_debug_schedule(n_heads, n, aq, ak, n_ctas_max, unit_pairs, rec, total, hdr)
    pieces = [tuple(rec[8 * i:8 * i + 8]) for i in range(total)]
    return dict(n_ctas=hdr[0], n_full=hdr[1], merge_pairs=hdr[2], iters_per_cta=hdr[3]), pieces


def ff_version() -> str:
    return load().ff_version().decode()


def ff_last_cuda_error() -> int:
    return load().ff_last_cuda_error()
