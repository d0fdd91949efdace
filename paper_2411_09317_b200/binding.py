"""ctypes binding of libpie.so: the same entry points as include/pie.h, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; nothing here computes.  Importing this module
loads the library and fails loudly (OSError) if it has not been built - there is no fallback.
Device arguments are raw addresses: pass ``tensor.data_ptr()`` of a CUDA tensor (or 0 / None for NULL);
host arrays are numpy arrays.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpie.so")
SYNTH_LIB_PATH = os.path.join(_HERE, "libpie_synth.so")

PIE_OK = 0
PIE_ERR_INVALID, PIE_ERR_RANGE, PIE_ERR_NOMEM, PIE_ERR_BUSY = -1, -2, -3, -4
PIE_ERR_NOT_RESIDENT, PIE_ERR_TIMEOUT, PIE_ERR_CUDA, PIE_ERR_UNSUPPORTED = -5, -6, -7, -8
PIE_F16, PIE_BF16 = 0, 1
PIE_MODE_AUTO, PIE_MODE_KERNEL, PIE_MODE_COPY_ENGINE, PIE_MODE_KERNEL_BULK = 0, 1, 2, 3
PIE_H2D, PIE_D2H = 0, 1
PIE_FREE, PIE_GPU, PIE_TO_HOST, PIE_HOST, PIE_TO_GPU = 0, 1, 2, 3, 4
PIE_Q_NONE, PIE_Q_IN, PIE_Q_OUT, PIE_Q_COMPUTE = 0, 1, 2, 3

EXPORTS = [
    "pie_pool_create", "pie_pool_destroy", "pie_block_bytes", "pie_block_alloc", "pie_block_free", "pie_block_write",
    "pie_block_read", "pie_block_state", "pie_get_placement", "pie_swap_out", "pie_swap_in", "pie_swap_raw",
    "pie_decode_attention", "pie_decode_step", "pie_decode_step_host", "pie_step_begin", "pie_set_extension_ratio",
    "pie_get_extension_ratio", "pie_set_controller", "pie_plan_layer", "pie_controller_tick", "pie_get_stats", "pie_get_step_timeline", "pie_sync", "pie_status_str",
    "pie_last_cuda_error", "pie_probe_link", "pie_probe_hbm", "pie_table_create", "pie_table_destroy", "pie_table_alloc",
    "pie_table_free", "pie_table_swap", "pie_table_attention", "pie_table_confirm", "pie_table_state", "pie_fifo_create",
    "pie_fifo_destroy", "pie_fifo_complete", "pie_fifo_layer_start", "pie_fifo_location", "pie_fifo_counters", "pie_layer_controller_decide", "pie_controller_decide",
    "pie_decode_attention_noalloc", "pie_set_layer_policy", "pie_set_violation_trigger", "pie_get_layer_log",
    "pie_resize_begin", "pie_resize_status", "pie_table_init_capacity", "pie_table_resize_begin", "pie_table_layer_pass",
    "pie_table_capacity", "pie_table_swap_ex", "pie_table_set_retention", "pie_table_kept_copies", "pie_table_mark_dirty", "pie_table_drop_host_copy", "pie_set_retention",
    "pie_declare_append_blocks", "pie_kv_write", "pie_prefill_attention", "pie_decode_layer", "pie_set_lookahead", "pie_set_run_ahead", "pie_set_kv_scales",
    "pie_governor_create", "pie_governor_destroy", "pie_governor_report", "pie_governor_state", "pie_report_throughput",
]


class PoolConfig(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("block_tokens", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("n_logical_blocks", ctypes.c_int32), ("max_seqs", ctypes.c_int32), ("own_streams", ctypes.c_int32),
        ("n_gpu_slots", ctypes.c_int64), ("n_host_slots", ctypes.c_int64),
        ("gpu_base", ctypes.c_void_p), ("host_base", ctypes.c_void_p),
        ("compute_stream", ctypes.c_void_p), ("copy_in_stream", ctypes.c_void_p), ("copy_out_stream", ctypes.c_void_p),
        ("split_tokens", ctypes.c_int32), ("swap_ctas", ctypes.c_int32),
        ("attn_ctas_per_sm", ctypes.c_int32), ("timing", ctypes.c_int32),
        ("attn_variant", ctypes.c_int32), ("visible_blocks", ctypes.c_int32), ("kv_format", ctypes.c_int32),
        ("reserved", ctypes.c_int32 * 5),
    ]


class Stats(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("governor_state", ctypes.c_uint32),
        ("bytes_in", ctypes.c_double), ("bytes_out", ctypes.c_double),
        ("calls_kernel", ctypes.c_double), ("calls_copy_engine", ctypes.c_double),
        ("last_step_compute_ms", ctypes.c_double), ("last_step_stall_ms", ctypes.c_double),
        ("last_step_swap_in_ms", ctypes.c_double), ("last_step_swap_out_ms", ctypes.c_double),
        ("last_step_ms", ctypes.c_double), ("ratio", ctypes.c_double),
        ("n_units_gpu", ctypes.c_int64), ("n_units_host", ctypes.c_int64), ("n_units_in_flight", ctypes.c_int64),
        ("steps_measured", ctypes.c_int64),
        ("last_step_slowdown_ms", ctypes.c_double), ("ratio_floor", ctypes.c_double), ("bytes_out_elided", ctypes.c_double),
        ("patch_kernel_launches", ctypes.c_double), ("governor_cap", ctypes.c_double),
        ("prefetch_lists", ctypes.c_int64), ("prefetch_violations", ctypes.c_int64),
        ("last_step_violation_ratio", ctypes.c_double), ("copy_engine_copies", ctypes.c_double),
        ("reserved", ctypes.c_double * 3),
    ]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_ if k not in ("reserved", "struct_size")}


lib = ctypes.CDLL(LIB_PATH)

_vp, _i32, _i64, _f32, _f64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_double
_sig = {
    "pie_pool_create": (_i32, [ctypes.POINTER(PoolConfig), ctypes.POINTER(_vp)]),
    "pie_pool_destroy": (_i32, [_vp]),
    "pie_block_bytes": (ctypes.c_size_t, [_vp]),
    "pie_block_alloc": (_i32, [_vp, _i64, _vp, _vp]),
    "pie_block_free": (_i32, [_vp, _vp, _i64]),
    "pie_block_write": (_i32, [_vp, _i32, _i32, _vp]),
    "pie_block_read": (_i32, [_vp, _i32, _i32, _vp]),
    "pie_block_state": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp]),
    "pie_get_placement": (_i32, [_vp, _vp, _vp]),
    "pie_swap_out": (_i32, [_vp, _i32, _vp, _i64, _i32]),
    "pie_swap_in": (_i32, [_vp, _i32, _vp, _i64, _i32]),
    "pie_swap_raw": (_i32, [_vp, _i32, _vp, _vp, _i64, _i32, _vp]),
    "pie_decode_attention": (_i32, [_vp, _i32, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _i32, _f32, _vp, _vp]),
    "pie_decode_step": (_i32, [_vp, _vp, _vp, _vp, _i32, _vp, _i32, _f32, _vp, _vp, _i32]),
    "pie_decode_step_host": (_i32, [_vp, _vp, _vp, _vp, _i32, _vp, _i32, _f32, _vp, _vp, _i32]),
    "pie_step_begin": (_i32, [_vp]),
    "pie_set_layer_policy": (_i32, [_vp, _i32, _i32]),
    "pie_get_layer_log": (_i32, [_vp, _vp, _i64, ctypes.POINTER(_i64)]),
    "pie_set_extension_ratio": (_i32, [_vp, _f32]),
    "pie_get_extension_ratio": (_i32, [_vp, ctypes.POINTER(_f32)]),
    "pie_set_controller": (_i32, [_vp, _f64, _f64, _f64]),
    "pie_plan_layer": (_i32, [_vp, _i32, _vp, ctypes.POINTER(_i64), _vp, ctypes.POINTER(_i64)]),
    "pie_controller_tick": (_i32, [_vp, ctypes.POINTER(_i32)]),
    "pie_get_stats": (_i32, [_vp, ctypes.POINTER(Stats)]),
    "pie_get_step_timeline": (_i32, [_vp, _vp, _i64]),
    "pie_sync": (_i32, [_vp, _i64]),
    "pie_status_str": (ctypes.c_char_p, [_i32]),
    "pie_last_cuda_error": (_i32, []),
    "pie_probe_link": (_i32, [_i64, _i32, _i32, ctypes.POINTER(_f64)]),
    "pie_probe_hbm": (_i32, [_i64, _i32, ctypes.POINTER(_f64)]),
    "pie_table_create": (_vp, [_i32, _i32, _i64, _i64]),
    "pie_table_destroy": (None, [_vp]),
    "pie_table_alloc": (_i32, [_vp, _i32, _i32]),
    "pie_table_free": (_i32, [_vp, _i32]),
    "pie_table_swap": (_i32, [_vp, _i32, _i32, _vp, _i64, ctypes.POINTER(_i64), _vp, _vp, _vp, ctypes.POINTER(_i64), _vp]),
    "pie_table_attention": (_i32, [_vp, _i32, _vp, _i64, ctypes.POINTER(_i64), _vp]),
    "pie_table_confirm": (_i32, [_vp, _i32, _i64]),
    "pie_table_state": (_i32, [_vp, _i32, _i32, ctypes.POINTER(_i32), ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "pie_table_swap_ex": (_i32, [_vp, _i32, _i32, _vp, _i64, ctypes.POINTER(_i64), _vp, _vp, _vp, _vp, ctypes.POINTER(_i64), _vp]),
    "pie_table_set_retention": (_i32, [_vp, _i32]),
    "pie_table_kept_copies": (_i64, [_vp]),
    "pie_table_mark_dirty": (_i32, [_vp, _i32, _vp, _i64]),
    "pie_table_drop_host_copy": (_i32, [_vp, _i32, _i32]),
    "pie_set_retention": (_i32, [_vp, _i32]),
    "pie_set_lookahead": (_i32, [_vp, _i32]),
    "pie_set_run_ahead": (_i32, [_vp, _i32]),
    "pie_set_kv_scales": (_i32, [_vp, ctypes.c_float, ctypes.c_float]),
    "pie_governor_create": (_vp, [_f64, _f64, _i32, _i32]),
    "pie_governor_destroy": (None, [_vp]),
    "pie_governor_report": (_f64, [_vp, _f64, _f64]),
    "pie_governor_state": (_i32, [_vp, _vp, _vp]),
    "pie_report_throughput": (_i32, [_vp, _f64]),
    "pie_decode_layer": (_i32, [_vp, _i32, _vp, _vp, _vp, _i32, _vp, _i32, _f32, _vp, _vp, _i32]),
    "pie_kv_write": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _i64, _vp, _i32, _i32]),
    "pie_declare_append_blocks": (_i32, [_vp, _vp, _i64]),
    "pie_table_init_capacity": (_i32, [_vp, _i32]),
    "pie_table_resize_begin": (_i32, [_vp, _i32]),
    "pie_table_layer_pass": (_i32, [_vp, _i32]),
    "pie_table_capacity": (_i32, [_vp] + [ctypes.POINTER(_i32)] * 4),
    "pie_resize_begin": (_i32, [_vp, _i32]),
    "pie_resize_status": (_i32, [_vp] + [ctypes.POINTER(_i32)] * 4),
    "pie_fifo_create": (_vp, [_i32, _i32, _i32, _vp]),
    "pie_fifo_destroy": (None, [_vp]),
    "pie_fifo_complete": (_i32, [_vp, _i32]),
    "pie_fifo_layer_start": (_i32, [_vp, _i32, ctypes.POINTER(_i32), ctypes.POINTER(_i32)]),
    "pie_fifo_location": (_i32, [_vp, _i32]),
    "pie_controller_decide": (_f64, [_vp, _f64, _f64, _f64, _f64, _f64]),
    "pie_set_violation_trigger": (_i32, [_vp, _f64]),
    "pie_prefill_attention": (_i32, [_vp, _i32, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _i32, _f32]),
    "pie_fifo_counters": (_i32, [_vp, ctypes.POINTER(_i64), ctypes.POINTER(_i64)]),
    "pie_layer_controller_decide": (_i32, [_vp, _i32, _i32, _f64, _f64, _i64, _i64, _f64, _f64]),
    "pie_decode_attention_noalloc": (_i32, [_vp, _i64, _vp, _i32, _vp, _vp, _vp, _i32, _vp, _vp, _i32, _i32, _i32, _i32, _i32,
                                            _i32, _f32, _vp, _vp]),
}
for _name, (_res, _args) in _sig.items():
    _fn = getattr(lib, _name)
    _fn.restype, _fn.argtypes = _res, _args


class PieError(RuntimeError):
    def __init__(self, status, where=""):
        self.status = status
        msg = lib.pie_status_str(status).decode()
        if status == PIE_ERR_CUDA:
            msg += f" (cudaError {lib.pie_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


def check(status, where=""):
    if status != PIE_OK:
        raise PieError(status, where)


def _np_i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a):
    """numpy array -> host address; int -> as is; None -> NULL"""
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return int(a)


# ---- pool ------------------------------------------------------------------------------------------------
def pie_pool_create(**kw) -> int:
    cfg = PoolConfig()
    kw.setdefault("block_tokens", 16)
    kw.setdefault("own_streams", 1)
    kw.setdefault("max_seqs", 256)
    cfg.struct_size = ctypes.sizeof(PoolConfig)
    cfg.attn_variant = kw.pop("attn_variant", 0)
    cfg.visible_blocks = kw.pop("visible_blocks", 0)
    cfg.kv_format = int(kw.pop("kv_fp8", 0))
    for k, v in kw.items():
        setattr(cfg, k, v)
    out = _vp()
    check(lib.pie_pool_create(ctypes.byref(cfg), ctypes.byref(out)), "pie_pool_create")
    return out.value


def pie_pool_destroy(pool) -> None:
    check(lib.pie_pool_destroy(pool), "pie_pool_destroy")


def pie_kv_write(pool, layer, k, v, token_seq_dev, token_pos_dev, n_tokens, block_table_dev, max_blocks_per_seq, n_seqs) -> None:
    check(lib.pie_kv_write(pool, layer, k, v, token_seq_dev, token_pos_dev, n_tokens, block_table_dev, max_blocks_per_seq,
                           n_seqs), "pie_kv_write")


def pie_prefill_attention(pool, layer, q, out, block_table_dev, max_blocks_per_seq, ctx_lens_dev, q_offsets_dev, ctx_lens_host,
                          q_offsets_host, n_seqs, scale) -> None:
    """q / out / *_dev: device pointers; ctx_lens_host [n_seqs], q_offsets_host [n_seqs + 1]: numpy int32."""
    ch, qh = _np_i32(ctx_lens_host), _np_i32(q_offsets_host)
    check(lib.pie_prefill_attention(pool, layer, q, out, block_table_dev, max_blocks_per_seq, ctx_lens_dev, q_offsets_dev, _ptr(ch),
                                    _ptr(qh), n_seqs, scale), "pie_prefill_attention")


def pie_set_violation_trigger(pool, share) -> None:
    check(lib.pie_set_violation_trigger(pool, share), "pie_set_violation_trigger")


def pie_set_lookahead(pool, layers) -> None:
    check(lib.pie_set_lookahead(pool, layers), "pie_set_lookahead")


def pie_set_run_ahead(pool, steps) -> None:
    check(lib.pie_set_run_ahead(pool, steps), "pie_set_run_ahead")


def pie_set_kv_scales(pool, k_scale, v_scale) -> None:
    check(lib.pie_set_kv_scales(pool, k_scale, v_scale), "pie_set_kv_scales")


def pie_report_throughput(pool, throughput) -> None:
    check(lib.pie_report_throughput(pool, throughput), "pie_report_throughput")


class Governor:
    """Throughput records (host only): report(ratio, throughput) -> cap on the ratio (1.0 = none)."""

    def __init__(self, step, tol=0.0, period=0, patience=0):
        self.h = lib.pie_governor_create(step, tol, period, patience)
        assert self.h

    def report(self, ratio, throughput) -> float:
        return lib.pie_governor_report(self.h, ratio, throughput)

    def state(self):
        s, c = np.zeros(1, np.int32), np.zeros(1, np.int32)
        check(lib.pie_governor_state(self.h, _ptr(s), _ptr(c)), "pie_governor_state")
        return int(s[0]), int(c[0])

    def close(self):
        if self.h:
            lib.pie_governor_destroy(self.h)
            self.h = None


def pie_set_retention(pool, on) -> None:
    check(lib.pie_set_retention(pool, int(on)), "pie_set_retention")


def pie_declare_append_blocks(pool, ids) -> None:
    if ids is None:
        check(lib.pie_declare_append_blocks(pool, None, -1), "pie_declare_append_blocks")
    else:
        ids = _np_i32(ids)
        check(lib.pie_declare_append_blocks(pool, _ptr(ids), len(ids)), "pie_declare_append_blocks")


def pie_resize_begin(pool, new_blocks) -> None:
    check(lib.pie_resize_begin(pool, new_blocks), "pie_resize_begin")


def pie_resize_status(pool) -> dict:
    v = [_i32() for _ in range(4)]
    check(lib.pie_resize_status(pool, *[ctypes.byref(x) for x in v]), "pie_resize_status")
    return dict(zip(("visible", "alloc_limit", "target", "layers_moved"), (x.value for x in v)))


def pie_block_bytes(pool) -> int:
    return int(lib.pie_block_bytes(pool))


def pie_block_alloc(pool, n, on_host=None) -> np.ndarray:
    ids = np.zeros(n, dtype=np.int32)
    flags = None if on_host is None else np.ascontiguousarray(on_host, dtype=np.uint8)
    check(lib.pie_block_alloc(pool, n, _ptr(flags), _ptr(ids)), "pie_block_alloc")
    return ids


def pie_block_free(pool, ids) -> None:
    ids = _np_i32(ids)
    check(lib.pie_block_free(pool, _ptr(ids), len(ids)), "pie_block_free")


def pie_block_write(pool, layer, block, data: np.ndarray) -> None:
    data = np.ascontiguousarray(data)
    assert data.nbytes == pie_block_bytes(pool)
    check(lib.pie_block_write(pool, layer, block, _ptr(data)), "pie_block_write")


def pie_block_read(pool, layer, block) -> np.ndarray:
    out = np.zeros(pie_block_bytes(pool), dtype=np.uint8)
    check(lib.pie_block_read(pool, layer, block, _ptr(out)), "pie_block_read")
    return out


def pie_block_state(pool, layer, block):
    s, g, h = np.zeros(1, np.int32), np.zeros(1, np.int32), np.zeros(1, np.int32)
    check(lib.pie_block_state(pool, layer, block, _ptr(s), _ptr(g), _ptr(h)), "pie_block_state")
    return int(s[0]), int(g[0]), int(h[0])


def pie_get_placement(pool, n_layers, n_logical):
    side = np.zeros((n_layers, n_logical), dtype=np.int32)
    slot = np.zeros((n_layers, n_logical), dtype=np.int32)
    check(lib.pie_get_placement(pool, _ptr(side), _ptr(slot)), "pie_get_placement")
    return side, slot


# ---- swapping ----------------------------------------------------------------------------------------------
def pie_swap_out(pool, layer, block_ids, mode=PIE_MODE_AUTO) -> None:
    ids = _np_i32(block_ids)
    check(lib.pie_swap_out(pool, layer, _ptr(ids), len(ids), mode), "pie_swap_out")


def pie_swap_in(pool, layer, block_ids, mode=PIE_MODE_AUTO) -> None:
    ids = _np_i32(block_ids)
    check(lib.pie_swap_in(pool, layer, _ptr(ids), len(ids), mode), "pie_swap_in")


def pie_swap_raw(pool, direction, src_slots, dst_slots, mode=PIE_MODE_KERNEL, stream=None) -> None:
    src, dst = _np_i32(src_slots), _np_i32(dst_slots)
    assert len(src) == len(dst)
    check(lib.pie_swap_raw(pool, direction, _ptr(src), _ptr(dst), len(src), mode, stream), "pie_swap_raw")


# ---- attention -----------------------------------------------------------------------------------------------
def pie_decode_attention(pool, layer, q, out, block_table_dev, max_blocks_per_seq, ctx_lens_dev, n_seqs, scale,
                         block_table_host=None, ctx_lens_host=None, k_new=None, v_new=None) -> None:
    bth = None if block_table_host is None else _np_i32(block_table_host)
    clh = None if ctx_lens_host is None else _np_i32(ctx_lens_host)
    check(lib.pie_decode_attention(pool, layer, _ptr(q), _ptr(out), _ptr(block_table_dev), max_blocks_per_seq,
                                   _ptr(ctx_lens_dev), _ptr(bth), _ptr(clh), n_seqs, scale, _ptr(k_new), _ptr(v_new)),
          "pie_decode_attention")


def pie_decode_step(pool, q_all, out_all, block_table_dev, max_blocks_per_seq, ctx_lens_dev, n_seqs, scale,
                    k_new_all=None, v_new_all=None, mode=PIE_MODE_AUTO) -> None:
    check(lib.pie_decode_step(pool, _ptr(q_all), _ptr(out_all), _ptr(block_table_dev), max_blocks_per_seq,
                              _ptr(ctx_lens_dev), n_seqs, scale, _ptr(k_new_all), _ptr(v_new_all), mode), "pie_decode_step")


def pie_decode_layer(pool, layer, q, out, block_table_dev, max_blocks_per_seq, ctx_lens_dev, n_seqs, scale, k_new=None,
                     v_new=None, mode=PIE_MODE_AUTO) -> None:
    check(lib.pie_decode_layer(pool, layer, _ptr(q), _ptr(out), _ptr(block_table_dev), max_blocks_per_seq, _ptr(ctx_lens_dev),
                               n_seqs, scale, _ptr(k_new), _ptr(v_new), mode), "pie_decode_layer")


def pie_decode_step_host(pool, q_all_host, out_all_host, block_table_host, max_blocks_per_seq, ctx_lens_host, n_seqs,
                         scale, k_new_all_host=None, v_new_all_host=None, mode=PIE_MODE_AUTO) -> None:
    check(lib.pie_decode_step_host(pool, _ptr(q_all_host), _ptr(out_all_host), _ptr(block_table_host), max_blocks_per_seq,
                                   _ptr(ctx_lens_host), n_seqs, scale, _ptr(k_new_all_host), _ptr(v_new_all_host), mode),
          "pie_decode_step_host")


def pie_set_layer_policy(pool, gpu_regions, cpu_regions) -> None:
    check(lib.pie_set_layer_policy(pool, gpu_regions, cpu_regions), "pie_set_layer_policy")


def pie_get_layer_log(pool) -> np.ndarray:
    n = _i64()
    check(lib.pie_get_layer_log(pool, None, 0, ctypes.byref(n)), "pie_get_layer_log")
    log = np.zeros((max(n.value, 1), 4), dtype=np.int32)
    check(lib.pie_get_layer_log(pool, _ptr(log), log.size, ctypes.byref(n)), "pie_get_layer_log")
    return log[:n.value]


def pie_step_begin(pool) -> None:
    check(lib.pie_step_begin(pool), "pie_step_begin")


# ---- policy / controller -----------------------------------------------------------------------------------
def pie_set_extension_ratio(pool, r: float) -> None:
    check(lib.pie_set_extension_ratio(pool, r), "pie_set_extension_ratio")


def pie_get_extension_ratio(pool) -> float:
    r = _f32()
    check(lib.pie_get_extension_ratio(pool, ctypes.byref(r)), "pie_get_extension_ratio")
    return r.value


def pie_set_controller(pool, step=0.0, eps=0.0, u_hi=0.0) -> None:
    check(lib.pie_set_controller(pool, step, eps, u_hi), "pie_set_controller")


def pie_plan_layer(pool, layer, n_logical):
    a, b = np.zeros(n_logical, np.int32), np.zeros(n_logical, np.int32)
    na, nb = _i64(), _i64()
    check(lib.pie_plan_layer(pool, layer, _ptr(a), ctypes.byref(na), _ptr(b), ctypes.byref(nb)), "pie_plan_layer")
    return a[:na.value].copy(), b[:nb.value].copy()


def pie_controller_tick(pool) -> bool:
    c = _i32()
    check(lib.pie_controller_tick(pool, ctypes.byref(c)), "pie_controller_tick")
    return bool(c.value)


def pie_get_stats(pool) -> dict:
    s = Stats()
    s.struct_size = ctypes.sizeof(Stats)
    check(lib.pie_get_stats(pool, ctypes.byref(s)), "pie_get_stats")
    return s.as_dict()


def pie_get_step_timeline(pool, n_layers) -> np.ndarray:
    out = np.zeros((n_layers, 7), dtype=np.float32)
    check(lib.pie_get_step_timeline(pool, _ptr(out), out.size), "pie_get_step_timeline")
    return out


def pie_sync(pool, timeout_us=60_000_000) -> None:
    check(lib.pie_sync(pool, timeout_us), "pie_sync")


def pie_probe_link(nbytes, direction, reps=3) -> float:
    g = _f64()
    check(lib.pie_probe_link(nbytes, direction, reps, ctypes.byref(g)), "pie_probe_link")
    return g.value


def pie_probe_hbm(nbytes, reps=3) -> float:
    g = _f64()
    check(lib.pie_probe_hbm(nbytes, reps, ctypes.byref(g)), "pie_probe_hbm")
    return g.value


def pie_decode_attention_noalloc(kv_pool, n_slots, slot_table, n_logical_blocks, q, out, block_table_dev,
                                 max_blocks_per_seq, ctx_lens_dev, ctx_lens_host, n_seqs, n_q_heads, n_kv_heads, head_dim,
                                 dtype, scale, split_tokens=0, status_dev=None, stream=None) -> None:
    """Attention for callers that may not allocate: no pool, the split-K scratch is a fixed device array inside
    the library (see include/pie.h).  All device arguments are raw addresses owned by the caller."""
    clh = _np_i32(ctx_lens_host)
    check(lib.pie_decode_attention_noalloc(_ptr(kv_pool), n_slots, _ptr(slot_table), n_logical_blocks, _ptr(q), _ptr(out),
                                           _ptr(block_table_dev), max_blocks_per_seq, _ptr(ctx_lens_dev), _ptr(clh), n_seqs,
                                           n_q_heads, n_kv_heads, head_dim, dtype, split_tokens, scale, _ptr(status_dev),
                                           _ptr(stream)), "pie_decode_attention_noalloc")


# ---- host-only pieces ------------------------------------------------------------------------------------------
class Table:
    """pie_table_* with numpy marshalling (the mapping table by itself; needs no GPU)."""

    def __init__(self, n_layers, n_logical, n_gpu_slots, n_host_slots):
        self.h = lib.pie_table_create(n_layers, n_logical, n_gpu_slots, n_host_slots)
        if not self.h:
            raise PieError(PIE_ERR_INVALID, "pie_table_create")

    def __del__(self):
        if getattr(self, "h", None):
            lib.pie_table_destroy(self.h)
            self.h = None

    def alloc(self, block, on_host=False):
        return lib.pie_table_alloc(self.h, block, int(on_host))

    def free(self, block):
        return lib.pie_table_free(self.h, block)

    def swap(self, queue, layer, ids):
        ids = _np_i32(ids)
        n = max(len(ids), 1)
        moved, src, dst = np.zeros(n, np.int32), np.zeros(n, np.int32), np.zeros(n, np.int32)
        elided = np.zeros(n, np.uint8)
        waits = np.zeros(4, np.int64)
        ticket, n_moved = _i64(), _i64()
        st = lib.pie_table_swap_ex(self.h, queue, layer, _ptr(ids), len(ids), ctypes.byref(ticket), _ptr(moved), _ptr(src),
                                   _ptr(dst), _ptr(elided), ctypes.byref(n_moved), _ptr(waits))
        k = n_moved.value if st == PIE_OK else 0
        pairs = [(int(moved[i]), int(src[i]), int(dst[i])) for i in range(k)]
        self.last_elided = [bool(elided[i]) for i in range(k)]   # pairs that need no bytes moved (kept host copies)
        return st, (ticket.value if st == PIE_OK else 0), pairs, {q: int(waits[q]) for q in range(1, 4) if waits[q]}

    def set_retention(self, on):
        return lib.pie_table_set_retention(self.h, int(on))

    def kept_copies(self):
        return int(lib.pie_table_kept_copies(self.h))

    def mark_dirty(self, layer, ids):
        ids = _np_i32(ids)
        return lib.pie_table_mark_dirty(self.h, layer, _ptr(ids), len(ids))

    def drop_host_copy(self, layer, block):
        return lib.pie_table_drop_host_copy(self.h, layer, block)

    def attention(self, layer, ids):
        waits = np.zeros(4, np.int64)
        ticket = _i64()
        if ids is None:
            st = lib.pie_table_attention(self.h, layer, None, 0, ctypes.byref(ticket), _ptr(waits))
        else:
            ids = _np_i32(ids)
            st = lib.pie_table_attention(self.h, layer, _ptr(ids), len(ids), ctypes.byref(ticket), _ptr(waits))
        return st, (ticket.value if st == PIE_OK else 0), {q: int(waits[q]) for q in range(1, 4) if waits[q]}

    def confirm(self, queue, ticket):
        return lib.pie_table_confirm(self.h, queue, ticket)

    def state(self, layer, block):
        s, g, h = _i32(), _i32(), _i32()
        st = lib.pie_table_state(self.h, layer, block, ctypes.byref(s), ctypes.byref(g), ctypes.byref(h))
        return st, s.value, g.value, h.value


    def init_capacity(self, size):
        return lib.pie_table_init_capacity(self.h, size)

    def resize_begin(self, new_size):
        return lib.pie_table_resize_begin(self.h, new_size)

    def layer_pass(self, layer):
        return lib.pie_table_layer_pass(self.h, layer)

    def capacity(self):
        v = [_i32() for _ in range(4)]
        st = lib.pie_table_capacity(self.h, *[ctypes.byref(x) for x in v])
        return st, dict(zip(("visible", "alloc_limit", "target", "layers_moved"), (x.value for x in v)))


class Fifo:
    """pie_fifo_*: the whole-layer swap protocol as a scheduler object (needs no GPU)."""

    def __init__(self, n_layers, gpu_regions, cpu_regions, on_cpu):
        flags = np.ascontiguousarray(on_cpu, dtype=np.uint8)
        self.h = lib.pie_fifo_create(n_layers, gpu_regions, cpu_regions, _ptr(flags))
        if not self.h:
            raise PieError(PIE_ERR_INVALID, "pie_fifo_create")

    def __del__(self):
        if getattr(self, "h", None):
            lib.pie_fifo_destroy(self.h)
            self.h = None

    def complete(self, direction):
        return lib.pie_fifo_complete(self.h, direction)

    def layer_start(self, k):
        o, i = _i32(), _i32()
        st = lib.pie_fifo_layer_start(self.h, k, ctypes.byref(o), ctypes.byref(i))
        return st, o.value, i.value

    def location(self, layer):
        return lib.pie_fifo_location(self.h, layer)

    def counters(self):
        """-> (swap-ins started, of which for a layer of the next token)"""
        a, b = _i64(), _i64()
        check(lib.pie_fifo_counters(self.h, ctypes.byref(a), ctypes.byref(b)), "pie_fifo_counters")
        return a.value, b.value


def pie_controller_decide(state: np.ndarray, ratio, step, stall, compute, swap_busy) -> float:
    assert state.dtype == np.float64 and state.size >= 8
    return lib.pie_controller_decide(_ptr(state), ratio, step, stall, compute, swap_busy)


def pie_layer_controller_decide(state: np.ndarray, m, m_max, stall, compute, in_starts, violations, v_trigger=0.0, eps=0.0) -> int:
    assert state.dtype == np.float64 and state.size >= 4
    return lib.pie_layer_controller_decide(_ptr(state), m, m_max, stall, compute, in_starts, violations, v_trigger, eps)


# ---- input generator kernels (separate library; inputs only) ---------------------------------------------------
_synth = None


def synth_lib():
    global _synth
    if _synth is None:
        _synth = ctypes.CDLL(SYNTH_LIB_PATH)
        _synth.pie_synth_fill_slots.restype = _i32
        _synth.pie_synth_fill_slots.argtypes = [_vp, _vp, _i64, _i64, ctypes.c_uint64, _i32, _f32, _vp]
        _synth.pie_synth_fill_slots_bytes.restype = _i32
        _synth.pie_synth_fill_slots_bytes.argtypes = [_vp, _vp, _i64, _i64, ctypes.c_uint64, _vp]
        _synth.pie_synth_fill_rows.restype = _i32
        _synth.pie_synth_fill_rows.argtypes = [_vp, _vp, _i64, _i64, ctypes.c_uint64, _i32, _f32, _vp]
        _synth.pie_synth_fill_tensor.restype = _i32
        _synth.pie_synth_fill_tensor.argtypes = [_vp, _i64, ctypes.c_uint64, ctypes.c_uint64, _i32, _f32, _vp]
    return _synth
