"""ctypes binding of include/adore.h. Argument marshalling only: every step runs in the library.

Functions carry the C names and take torch tensors (their data pointers are passed on) or
raw integer addresses. A status other than ADORE_OK raises AdoreError. The library must have
been built (python -m paper_2407_02328_b200.build); there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libadore.so")

ADORE_F32, ADORE_BF16 = 0, 1
ADORE_REBUILD_POLICY, ADORE_REBUILD_EXPLICIT = 0, 1
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "OOM", 3: "TOKEN_TABLE_FULL", 4: "STATE", 5: "CUDA",
                6: "DEVICE_FLAG", 7: "TIMEOUT", 8: "UNSUPPORTED"}


ADORE_FLAG_NO_RECURRENCE = 1
ADORE_FLAG_SCORE_FROM_ATTENTION = 2
ADORE_FLAG_RELATIVE_POSITION = 4


class AdoreError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({_lib().adore_status_string(status).decode()})")


class adore_config_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("batch", C.c_int32), ("n_layers", C.c_int32),
                ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("hidden", C.c_int32),
                ("capacity", C.c_int32), ("rebuild_max", C.c_int32), ("topk", C.c_int32),
                ("max_tokens", C.c_int32), ("ctrl_hidden", C.c_int32), ("dtype", C.c_int),
                ("rebuild_mode", C.c_int), ("rope_theta", C.c_float), ("pos_scale", C.c_float),
                ("flags", C.c_uint32)]


class adore_controller_weights_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("gru_w_ih", "gru_w_hh", "gru_b_ih", "gru_b_hh", "pos_w", "pos_b",
                                          "mlp_w1", "mlp_b1", "mlp_w2", "mlp_b2")]


_LIB = None
EXPORTS = ["adore_cache_create", "adore_cache_destroy", "adore_cache_set_projection",
           "adore_cache_append_tokens", "adore_cache_fill_layer", "adore_decode_step",
           "adore_decode_step_host", "adore_rebuild", "adore_cache_slot_map", "adore_cache_rebuild_list",
           "adore_cache_step_info", "adore_cache_scores", "adore_cache_kv", "adore_cache_num_tokens",
           "adore_cache_launch_count", "adore_cache_sync_status", "adore_cache_join", "adore_status_string",
           "adore_cache_set_stage_timing", "adore_cache_stage_times", "adore_cache_group_times", "adore_cache_rebuild_rows",
           "adore_controller_score_static",
           "adore_cache_export_state", "adore_cache_import_state", "adore_step_begin", "adore_attend_rows",
           "adore_label_tokens", "adore_decode_rebuild_host", "adore_decode_rebuild_host_queued", "adore_cache_wait_outputs"]


def _lib():
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2407_02328_b200.build`")
        lib = C.CDLL(LIB_PATH)
        vp, i32 = C.c_void_p, C.c_int32
        lib.adore_status_string.restype = C.c_char_p
        lib.adore_status_string.argtypes = [C.c_int]
        lib.adore_cache_create.argtypes = [C.POINTER(adore_config_t), C.POINTER(adore_controller_weights_t), vp, C.POINTER(vp)]
        lib.adore_cache_destroy.argtypes = [vp]
        lib.adore_cache_set_projection.argtypes = [vp, i32, vp]
        lib.adore_cache_append_tokens.argtypes = [vp, vp, i32]
        lib.adore_cache_fill_layer.argtypes = [vp, i32, vp]
        step = [vp, i32, vp, vp, vp, vp, vp, vp, i32, vp, vp]
        lib.adore_decode_step.argtypes = step
        lib.adore_decode_step_host.argtypes = step
        lib.adore_decode_rebuild_host.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
        lib.adore_decode_rebuild_host_queued.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
        lib.adore_rebuild.argtypes = [vp, i32, vp]
        lib.adore_step_begin.argtypes = [vp, vp, vp, vp, i32]
        lib.adore_label_tokens.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        lib.adore_attend_rows.argtypes = [vp, i32, vp, vp, vp, vp, vp]
        lib.adore_cache_slot_map.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
        lib.adore_cache_rebuild_list.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)]
        lib.adore_cache_step_info.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
        lib.adore_cache_scores.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
        lib.adore_cache_kv.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp)]
        lib.adore_cache_num_tokens.argtypes = [vp]
        lib.adore_cache_num_tokens.restype = i32
        lib.adore_cache_launch_count.argtypes = [vp]
        lib.adore_cache_launch_count.restype = C.c_int64
        lib.adore_cache_sync_status.argtypes = [vp]
        lib.adore_cache_join.argtypes = [vp]
        lib.adore_cache_wait_outputs.argtypes = [vp]
        lib.adore_cache_set_stage_timing.argtypes = [vp, i32]
        lib.adore_cache_stage_times.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        lib.adore_cache_group_times.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        lib.adore_cache_rebuild_rows.argtypes = [vp, C.POINTER(C.c_int64)]
        lib.adore_cache_export_state.argtypes = [vp, vp, C.POINTER(C.c_size_t)]
        lib.adore_cache_import_state.argtypes = [vp, vp, C.c_size_t]
        lib.adore_controller_score_static.argtypes = [C.POINTER(adore_controller_weights_t), C.c_int, i32, i32, i32, vp, vp,
                                                      i32, C.c_float, vp, vp, vp]
        _LIB = lib
    return _LIB


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert t.is_contiguous()
    return t.data_ptr()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise AdoreError(status, where)


def adore_cache_create(cfg: adore_config_t, ctrl: Dict[str, np.ndarray], cuda_stream: int = 0) -> int:
    keep = {k: np.ascontiguousarray(v, dtype=np.float32) for k, v in ctrl.items()}
    w = adore_controller_weights_t(**{k: keep[k].ctypes.data for k, _ in adore_controller_weights_t._fields_})
    out = C.c_void_p()
    cfg.struct_size = C.sizeof(adore_config_t)
    _check(_lib().adore_cache_create(C.byref(cfg), C.byref(w), cuda_stream or None, C.byref(out)), "adore_cache_create")
    return out.value


def adore_cache_destroy(cache: Optional[int]) -> None:
    _check(_lib().adore_cache_destroy(cache), "adore_cache_destroy")


def adore_cache_set_projection(cache: int, layer: int, w_kv) -> None:
    _check(_lib().adore_cache_set_projection(cache, layer, _ptr(w_kv)), "adore_cache_set_projection")


def adore_cache_append_tokens(cache: int, x, T: int) -> None:
    _check(_lib().adore_cache_append_tokens(cache, _ptr(x), T), "adore_cache_append_tokens")


def adore_cache_fill_layer(cache: int, layer: int, x_table=None) -> None:
    _check(_lib().adore_cache_fill_layer(cache, layer, _ptr(x_table)), "adore_cache_fill_layer")


def adore_decode_step(cache: int, layer: int, q, k_new, v_new, x_new, explicit_list, explicit_count, r_in: int,
                      out, weights=None) -> None:
    _check(_lib().adore_decode_step(cache, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(x_new), _ptr(explicit_list),
                                    _ptr(explicit_count), r_in, _ptr(out), _ptr(weights)), "adore_decode_step")


def adore_decode_step_host(cache: int, layer: int, q, k_new, v_new, x_new, explicit_list, explicit_count, r_in: int,
                           out, weights=None) -> None:
    _check(_lib().adore_decode_step_host(cache, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(x_new),
                                         _ptr(explicit_list), _ptr(explicit_count), r_in, _ptr(out), _ptr(weights)),
           "adore_decode_step_host")


def adore_decode_rebuild_host(cache: int, layer: int, q, k_new, v_new, x_new, explicit_list, explicit_count, r_in: int,
                              x_table, out, weights=None) -> None:
    _check(_lib().adore_decode_rebuild_host(cache, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(x_new),
                                            _ptr(explicit_list), _ptr(explicit_count), r_in, _ptr(x_table), _ptr(out),
                                            _ptr(weights)), "adore_decode_rebuild_host")


def adore_decode_rebuild_host_queued(cache: int, layer: int, q, k_new, v_new, x_new, explicit_list, explicit_count,
                                     r_in: int, x_table, out, weights=None) -> None:
    _check(_lib().adore_decode_rebuild_host_queued(cache, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(x_new),
                                                   _ptr(explicit_list), _ptr(explicit_count), r_in, _ptr(x_table), _ptr(out),
                                                   _ptr(weights)), "adore_decode_rebuild_host_queued")


def adore_step_begin(cache: int, x_new, explicit_list, explicit_count, r_in: int) -> None:
    _check(_lib().adore_step_begin(cache, _ptr(x_new), _ptr(explicit_list), _ptr(explicit_count), r_in), "adore_step_begin")


def adore_attend_rows(cache: int, layer: int, q_rows, k_new, v_new, out, weights=None) -> None:
    _check(_lib().adore_attend_rows(cache, layer, _ptr(q_rows), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(weights)),
           "adore_attend_rows")


def adore_label_tokens(weights, n_layers: int, batch: int, n_heads: int, n_slots: int, topk: int, cuda_stream: int,
                       sets, count, label, coverage, mass) -> None:
    _check(_lib().adore_label_tokens(_ptr(weights), n_layers, batch, n_heads, n_slots, topk, cuda_stream or None, _ptr(sets),
                                     _ptr(count), _ptr(label), _ptr(coverage), _ptr(mass)), "adore_label_tokens")


def adore_rebuild(cache: int, layer: int, x_table=None) -> None:
    _check(_lib().adore_rebuild(cache, layer, _ptr(x_table)), "adore_rebuild")


def _views(fn, cache: int, n: int, *extra) -> Tuple[int, ...]:
    outs = [C.c_void_p() for _ in range(n)]
    _check(fn(cache, *extra, *[C.byref(o) for o in outs]), fn.__name__)
    return tuple(o.value for o in outs)


def adore_cache_slot_map(cache: int) -> Tuple[int, int]:
    return _views(_lib().adore_cache_slot_map, cache, 2)


def adore_cache_rebuild_list(cache: int) -> Tuple[int, int, int]:
    return _views(_lib().adore_cache_rebuild_list, cache, 3)


def adore_cache_step_info(cache: int) -> Tuple[int, int]:
    return _views(_lib().adore_cache_step_info, cache, 2)


def adore_cache_scores(cache: int) -> Tuple[int, int]:
    return _views(_lib().adore_cache_scores, cache, 2)


def adore_cache_kv(cache: int, layer: int) -> Tuple[int, int]:
    return _views(_lib().adore_cache_kv, cache, 2, layer)


def adore_cache_num_tokens(cache: int) -> int:
    return _lib().adore_cache_num_tokens(cache)


def adore_cache_launch_count(cache: int) -> int:
    return _lib().adore_cache_launch_count(cache)


def adore_cache_join(cache: int) -> None:
    _check(_lib().adore_cache_join(cache), "adore_cache_join")


def adore_cache_wait_outputs(cache: int) -> None:
    _check(_lib().adore_cache_wait_outputs(cache), "adore_cache_wait_outputs")


def adore_cache_sync_status(cache: int) -> None:
    _check(_lib().adore_cache_sync_status(cache), "adore_cache_sync_status")


def adore_cache_export_state(cache: int, host_buf: Optional[np.ndarray] = None) -> int:
    """Bytes needed (host_buf None) or written into the uint8 array host_buf."""
    n = C.c_size_t(0 if host_buf is None else host_buf.nbytes)
    _check(_lib().adore_cache_export_state(cache, _ptr(host_buf), C.byref(n)), "adore_cache_export_state")
    return int(n.value)


def adore_cache_import_state(cache: int, host_buf: np.ndarray) -> None:
    _check(_lib().adore_cache_import_state(cache, _ptr(host_buf), host_buf.nbytes), "adore_cache_import_state")


def adore_cache_set_stage_timing(cache: int, enable) -> None:
    """enable: 0/False off, 1/True per-stage timing, 2 group timing."""
    _check(_lib().adore_cache_set_stage_timing(cache, int(enable)), "adore_cache_set_stage_timing")


def adore_cache_group_times(cache: int):
    """Returns (ms, ms_main, steps): device time of the attention + selection group summed over the steps since the last
    call, to the later of {main-stream part, controller chain} and to the end of the main-stream part alone."""
    ms, ms_main, n = C.c_double(), C.c_double(), C.c_int64()
    _check(_lib().adore_cache_group_times(cache, C.byref(ms), C.byref(ms_main), C.byref(n)), "adore_cache_group_times")
    return ms.value, ms_main.value, n.value


def adore_cache_stage_times(cache: int):
    """Returns ([ms attention, controller+select, rebuild, layer-0 admit], [launch counts]) since the last call."""
    ms = (C.c_double * 4)()
    n = (C.c_int64 * 4)()
    _check(_lib().adore_cache_stage_times(cache, ms, n), "adore_cache_stage_times")
    return list(ms), list(n)


def adore_cache_rebuild_rows(cache: int) -> int:
    v = C.c_int64()
    _check(_lib().adore_cache_rebuild_rows(cache, C.byref(v)), "adore_cache_rebuild_rows")
    return v.value


def adore_controller_score_static(weights_dev: Dict[str, object], dtype: str, batch: int, hidden: int, ctrl_hidden: int,
                                  x, z, position: int, pos_scale: float, score, sigma, cuda_stream: int = 0) -> None:
    """Scores one new token per sequence without any allocation; `weights_dev` maps the parameter
    names of adore_controller_weights_t to float32 CUDA tensors (or raw device addresses)."""
    w = adore_controller_weights_t(**{k: _ptr(weights_dev[k]) for k, _ in adore_controller_weights_t._fields_})
    _check(_lib().adore_controller_score_static(C.byref(w), ADORE_F32 if dtype == "f32" else ADORE_BF16, batch, hidden,
                                                ctrl_hidden, _ptr(x), _ptr(z), position, pos_scale, _ptr(score),
                                                _ptr(sigma), cuda_stream or None), "adore_controller_score_static")


def adore_status_string(status: int) -> str:
    return _lib().adore_status_string(status).decode()


# ---- helpers for harnesses: copy a device view into a torch tensor -----------------------------
class _RawDevice:
    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False), "version": 2}


def device_view(ptr: int, shape, dtype):
    """Wraps a raw device address as a torch CUDA tensor (no copy). dtype is a torch dtype."""
    import torch
    typestr = {torch.int32: "<i4", torch.uint8: "|u1", torch.float32: "<f4", torch.float64: "<f8",
               torch.bfloat16: "<u2"}[dtype]
    t = torch.as_tensor(_RawDevice(ptr, shape, typestr), device="cuda")
    return t.view(torch.bfloat16) if dtype == torch.bfloat16 else t


def make_config(*, batch, n_layers, n_heads, head_dim, hidden, capacity, rebuild_max, topk, max_tokens,
                ctrl_hidden=128, dtype="bf16", rebuild_mode="policy", rope_theta=1.0e4, pos_scale=4096.0,
                flags=0) -> adore_config_t:
    return adore_config_t(struct_size=C.sizeof(adore_config_t), batch=batch, n_layers=n_layers, n_heads=n_heads,
                          head_dim=head_dim, hidden=hidden, capacity=capacity, rebuild_max=rebuild_max, topk=topk,
                          max_tokens=max_tokens, ctrl_hidden=ctrl_hidden,
                          dtype=ADORE_F32 if dtype == "f32" else ADORE_BF16,
                          rebuild_mode=ADORE_REBUILD_POLICY if rebuild_mode == "policy" else ADORE_REBUILD_EXPLICIT,
                          rope_theta=rope_theta, pos_scale=pos_scale, flags=flags)
