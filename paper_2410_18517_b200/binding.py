"""ctypes binding of ``libkvs.so`` (the C ABI in ``include/kvs.h``).

Argument marshalling only: every function has the name of the C entry point it
calls and passes raw pointers, sizes and a CUDA stream handle.  Nothing here
computes anything; if the compiled library is missing the import of a function
fails loudly -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
# KVS_LIBRARY names another build of the same library (the bounds-checking one, for instance)
LIB_PATH = os.environ.get("KVS_LIBRARY") or os.path.join(_HERE, "libkvs.so")

KVS_OK = 0
KVS_ERR_INVALID_ARG = 1
KVS_ERR_BAD_SHARE_MAP = 2
KVS_ERR_STATE = 3
KVS_ERR_CAPACITY = 4
KVS_ERR_OOM = 5
KVS_ERR_CUDA = 6
KVS_ERR_TIMEOUT = 7
KVS_ERR_SCRATCH_LIMIT = 8
KVS_ERR_BOUNDS = 9

KVS_BF16 = 0
KVS_F32 = 1

KVS_OPT_MAX_CTAS = 0
KVS_OPT_KERNEL = 1
KVS_OPT_EARLY_START = 2
KVS_OPT_REPLAY = 3
KVS_OPT_HOST_CHUNKS = 4
KVS_OPT_FINISH_IN_KERNEL = 5
KVS_OPT_WAIT_LIMIT_US = 6

# every symbol include/kvs.h declares
EXPORTS = (
    "kvs_create", "kvs_destroy", "kvs_set_share_map", "kvs_required_bytes", "kvs_bind_memory",
    "kvs_reset", "kvs_append", "kvs_decode_attention", "kvs_step_host", "kvs_num_slots",
    "kvs_slot_of_layer", "kvs_seq_len", "kvs_row_stride", "kvs_plane_offset", "kvs_stats",
    "kvs_last_device_status", "kvs_set_option", "kvs_last_launch", "kvs_status_string",
    "kvs_read_roof", "kvs_decode_attention_static", "kvs_prefill_attention",
    "kvs_evict", "kvs_unit_len", "kvs_layer_distances", "kvs_mean_cosine",
    "kvs_replay_advance", "kvs_replay_commit", "kvs_decode_step",
    "kvs_clear_device_status", "kvs_selftest_wait_timeout", "kvs_truncate",
    "kvs_selftest_bounds", "kvs_selftest_stalled_copy", "kvs_trace_begin", "kvs_trace_end",
)


class kvs_config(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("max_batch", ctypes.c_int32), ("max_seq", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("softmax_scale", ctypes.c_float), ("device", ctypes.c_int32),
    ]


class kvs_stats_t(ctypes.Structure):
    _fields_ = [
        ("append_launches", ctypes.c_uint64), ("append_skipped", ctypes.c_uint64),
        ("attention_launches", ctypes.c_uint64), ("combine_launches", ctypes.c_uint64),
        ("kv_bytes_read", ctypes.c_uint64), ("kv_bytes_appended", ctypes.c_uint64),
        ("prefill_launches", ctypes.c_uint64), ("evict_launches", ctypes.c_uint64),
        ("search_launches", ctypes.c_uint64), ("fused_appends", ctypes.c_uint64),
    ]


_lib = None


def load() -> ctypes.CDLL:
    """Load the compiled library; raise if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2410_18517_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    P = ctypes.POINTER
    sig = {
        "kvs_create": [P(kvs_config), P(vp)],
        "kvs_destroy": [vp],
        "kvs_set_share_map": [vp, P(i32)],
        "kvs_required_bytes": [vp, P(sz), P(sz)],
        "kvs_bind_memory": [vp, vp, sz, vp, sz],
        "kvs_reset": [vp],
        "kvs_truncate": [vp, i32],
        "kvs_append": [vp, i32, vp, vp, i32, i32, vp],
        "kvs_decode_attention": [vp, i32, vp, vp, i32, vp],
        "kvs_decode_step": [vp, i32, vp, vp, vp, vp, i32, vp],
        "kvs_decode_attention_static": [vp, i32, vp, vp, i32, vp, vp],
        "kvs_prefill_attention": [vp, i32, vp, vp, i32, i32, vp],
        "kvs_evict": [vp, i32, vp, P(i32), i32, i32, vp],
        "kvs_unit_len": [vp, i32, i32, i32, P(i32)],
        "kvs_replay_advance": [vp, vp],
        "kvs_replay_commit": [vp, i32, vp],
        "kvs_layer_distances": [vp, i32, vp, vp],
        "kvs_mean_cosine": [vp, vp, vp, i32, ctypes.c_int64, vp, vp],
        "kvs_step_host": [vp, vp, vp, vp, vp, i32, vp, P(ctypes.c_uint64), P(ctypes.c_uint64)],
        "kvs_num_slots": [vp, P(i32)],
        "kvs_slot_of_layer": [vp, i32, P(i32)],
        "kvs_seq_len": [vp, i32, P(i32)],
        "kvs_row_stride": [vp, P(i32)],
        "kvs_plane_offset": [vp, i32, i32, P(sz)],
        "kvs_stats": [vp, P(kvs_stats_t)],
        "kvs_last_device_status": [vp, P(i32)],
        "kvs_clear_device_status": [vp, vp],
        "kvs_selftest_wait_timeout": [vp, ctypes.c_uint32, P(ctypes.c_uint64), vp],
        "kvs_selftest_bounds": [vp, vp],
        "kvs_trace_begin": [vp, vp, sz],
        "kvs_trace_end": [vp, P(i32)],
        "kvs_selftest_stalled_copy": [vp, i32, vp, vp, i32, vp],
        "kvs_set_option": [vp, i32, i32],
        "kvs_last_launch": [vp, P(i32), P(i32), P(i32)],
        "kvs_read_roof": [vp, sz, vp, i32, vp],
    }
    for name, argtypes in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = argtypes
        fn.restype = ctypes.c_int
    lib.kvs_status_string.argtypes = [ctypes.c_int]
    lib.kvs_status_string.restype = ctypes.c_char_p
    _lib = lib
    return lib


class KvsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {kvs_status_string(status)} (status {status})")


def _check(status: int, where: str) -> None:
    if status != KVS_OK:
        raise KvsError(status, where)


def _ptr(x) -> int | None:
    """Raw address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return x.ctypes.data


def kvs_status_string(status: int) -> str:
    return load().kvs_status_string(status).decode()


def kvs_create(n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_seq, dtype, softmax_scale=0.0,
               device=0) -> int:
    cfg = kvs_config(n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_seq, dtype, softmax_scale, device)
    h = ctypes.c_void_p()
    _check(load().kvs_create(ctypes.byref(cfg), ctypes.byref(h)), "kvs_create")
    return h.value


def kvs_destroy(ctx: int) -> None:
    _check(load().kvs_destroy(ctx), "kvs_destroy")


def kvs_set_share_map(ctx: int, share_map) -> None:
    arr = (ctypes.c_int32 * len(share_map))(*[int(x) for x in share_map])
    _check(load().kvs_set_share_map(ctx, arr), "kvs_set_share_map")


def kvs_required_bytes(ctx: int) -> tuple[int, int]:
    a, b = ctypes.c_size_t(), ctypes.c_size_t()
    _check(load().kvs_required_bytes(ctx, ctypes.byref(a), ctypes.byref(b)), "kvs_required_bytes")
    return a.value, b.value


def kvs_bind_memory(ctx: int, pool, pool_bytes: int, workspace, workspace_bytes: int) -> None:
    _check(load().kvs_bind_memory(ctx, _ptr(pool), pool_bytes, _ptr(workspace), workspace_bytes), "kvs_bind_memory")


def kvs_reset(ctx: int) -> None:
    _check(load().kvs_reset(ctx), "kvs_reset")


def kvs_truncate(ctx: int, n_tokens: int) -> None:
    _check(load().kvs_truncate(ctx, n_tokens), "kvs_truncate")


def kvs_append(ctx: int, layer: int, k, v, batch: int, n_new: int, stream: int = 0) -> None:
    _check(load().kvs_append(ctx, layer, _ptr(k), _ptr(v), batch, n_new, stream), "kvs_append")


def kvs_decode_attention(ctx: int, layer: int, q, out, batch: int, stream: int = 0) -> None:
    _check(load().kvs_decode_attention(ctx, layer, _ptr(q), _ptr(out), batch, stream), "kvs_decode_attention")


def kvs_decode_step(ctx: int, layer: int, q, k, v, out, batch: int, stream: int = 0) -> None:
    _check(load().kvs_decode_step(ctx, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(out), batch, stream), "kvs_decode_step")


def kvs_prefill_attention(ctx: int, layer: int, q, out, batch: int, n_q: int, stream: int = 0) -> None:
    _check(load().kvs_prefill_attention(ctx, layer, _ptr(q), _ptr(out), batch, n_q, stream), "kvs_prefill_attention")


def kvs_evict(ctx: int, layer: int, keep, n_keep, keep_stride: int, batch: int, stream: int = 0) -> None:
    """keep: device int32 ``[batch][Hkv][keep_stride]``; n_keep: host sequence of batch*Hkv counts."""
    counts = (ctypes.c_int32 * len(n_keep))(*[int(x) for x in n_keep])
    _check(load().kvs_evict(ctx, layer, _ptr(keep), counts, keep_stride, batch, stream), "kvs_evict")


def kvs_unit_len(ctx: int, layer: int, b: int, h: int) -> int:
    v = ctypes.c_int32()
    _check(load().kvs_unit_len(ctx, layer, b, h, ctypes.byref(v)), "kvs_unit_len")
    return v.value


def kvs_layer_distances(ctx: int, batch: int, dist, stream: int = 0) -> None:
    _check(load().kvs_layer_distances(ctx, batch, _ptr(dist), stream), "kvs_layer_distances")


def kvs_mean_cosine(ctx: int, a, b, n_samples: int, dim: int, out, stream: int = 0) -> None:
    _check(load().kvs_mean_cosine(ctx, _ptr(a), _ptr(b), n_samples, dim, _ptr(out), stream), "kvs_mean_cosine")


def kvs_replay_advance(ctx: int, stream: int = 0) -> None:
    _check(load().kvs_replay_advance(ctx, stream), "kvs_replay_advance")


def kvs_replay_commit(ctx: int, times_run: int, stream: int = 0) -> None:
    _check(load().kvs_replay_commit(ctx, times_run, stream), "kvs_replay_commit")


def kvs_decode_attention_static(ctx: int, layer: int, q, out, batch: int, stream: int = 0, device_status=None) -> None:
    """Same result as ``kvs_decode_attention``; scratch is the library's built-in 2 MiB array (no allocation)."""
    _check(load().kvs_decode_attention_static(ctx, layer, _ptr(q), _ptr(out), batch, stream, _ptr(device_status)),
           "kvs_decode_attention_static")


def kvs_step_host(ctx: int, q_host, k_host, v_host, out_host, batch: int, stream: int = 0) -> tuple[int, int]:
    h2d, d2h = ctypes.c_uint64(), ctypes.c_uint64()
    _check(load().kvs_step_host(ctx, _ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(out_host), batch, stream,
                                ctypes.byref(h2d), ctypes.byref(d2h)), "kvs_step_host")
    return h2d.value, d2h.value


def kvs_num_slots(ctx: int) -> int:
    v = ctypes.c_int32()
    _check(load().kvs_num_slots(ctx, ctypes.byref(v)), "kvs_num_slots")
    return v.value


def kvs_slot_of_layer(ctx: int, layer: int) -> int:
    v = ctypes.c_int32()
    _check(load().kvs_slot_of_layer(ctx, layer, ctypes.byref(v)), "kvs_slot_of_layer")
    return v.value


def kvs_seq_len(ctx: int, layer: int) -> int:
    v = ctypes.c_int32()
    _check(load().kvs_seq_len(ctx, layer, ctypes.byref(v)), "kvs_seq_len")
    return v.value


def kvs_row_stride(ctx: int) -> int:
    v = ctypes.c_int32()
    _check(load().kvs_row_stride(ctx, ctypes.byref(v)), "kvs_row_stride")
    return v.value


def kvs_plane_offset(ctx: int, slot: int, kv: int) -> int:
    v = ctypes.c_size_t()
    _check(load().kvs_plane_offset(ctx, slot, kv, ctypes.byref(v)), "kvs_plane_offset")
    return v.value


def kvs_stats(ctx: int) -> dict:
    s = kvs_stats_t()
    _check(load().kvs_stats(ctx, ctypes.byref(s)), "kvs_stats")
    return {name: int(getattr(s, name)) for name, _ in kvs_stats_t._fields_}


def kvs_last_device_status(ctx: int) -> int:
    v = ctypes.c_int32()
    _check(load().kvs_last_device_status(ctx, ctypes.byref(v)), "kvs_last_device_status")
    return v.value


def kvs_clear_device_status(ctx: int, stream: int = 0) -> None:
    _check(load().kvs_clear_device_status(ctx, stream), "kvs_clear_device_status")


def kvs_selftest_wait_timeout(ctx: int, limit_us: int, stream: int = 0) -> int:
    """Returns the nanoseconds the wait lasted on the GPU before it gave up."""
    w = ctypes.c_uint64()
    _check(load().kvs_selftest_wait_timeout(ctx, limit_us, ctypes.byref(w), stream), "kvs_selftest_wait_timeout")
    return w.value


def kvs_trace_begin(ctx: int, buffer, nbytes: int) -> None:
    _check(load().kvs_trace_begin(ctx, _ptr(buffer), nbytes), "kvs_trace_begin")


def kvs_trace_end(ctx: int) -> int:
    """Stops the recording; returns the number of attention calls recorded."""
    n = ctypes.c_int32()
    _check(load().kvs_trace_end(ctx, ctypes.byref(n)), "kvs_trace_end")
    return n.value


def kvs_selftest_bounds(ctx: int, stream: int = 0) -> None:
    _check(load().kvs_selftest_bounds(ctx, stream), "kvs_selftest_bounds")


def kvs_selftest_stalled_copy(ctx: int, layer: int, q, out, batch: int, stream: int = 0) -> None:
    _check(load().kvs_selftest_stalled_copy(ctx, layer, _ptr(q), _ptr(out), batch, stream), "kvs_selftest_stalled_copy")


def kvs_set_option(ctx: int, option: int, value: int) -> None:
    _check(load().kvs_set_option(ctx, option, value), "kvs_set_option")


def kvs_last_launch(ctx: int) -> dict:
    a, b, c = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(load().kvs_last_launch(ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)), "kvs_last_launch")
    return {"ctas": a.value, "tile_rows": b.value, "kernel": c.value}


def kvs_read_roof(src, nbytes: int, checksum, device: int = 0, stream: int = 0) -> None:
    _check(load().kvs_read_roof(_ptr(src), nbytes, _ptr(checksum), device, stream), "kvs_read_roof")
