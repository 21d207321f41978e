"""ctypes binding of libpreserve_b200.so: argument marshalling only.

Every function has the name and the argument order of its C declaration in
include/preserve_b200.h.  Tensors are passed as device pointers; the stream is torch's
current stream.  There is no fallback: if the library is missing, importing fails.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpreserve_b200.so")

PRE_OK, PRE_EINVAL, PRE_ECAPACITY, PRE_EBADREQ, PRE_ETIMEOUT, PRE_ECUDA, PRE_ENOMEM, PRE_ESIZE = 0, -1, -2, -3, -4, -5, -6, -7

EXPORTS = ("pre_create", "pre_destroy", "pre_anticipate", "pre_route_batch", "pre_step", "pre_status",
           "pre_last_cuda_error", "pre_strerror", "pre_query", "pre_anticipate_static", "pre_scaler_signals",
           "pre_refine", "pre_route_admit", "pre_ring_window", "pre_ring_fold", "pre_ring_step",
           "pre_ring_refine", "pre_test_set_spin_limit", "pre_query_layout", "pre_tick", "pre_route_select")


class pre_config(C.Structure):
    _fields_ = [("n_instances", C.c_int32), ("horizon", C.c_int32), ("capacity_tokens", C.c_int64),
                ("t_mem", C.c_double), ("beta", C.c_double), ("max_requests", C.c_int64)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2504_03702_b200.build` "
            "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i64 = C.c_void_p, C.c_int64
    lib.pre_create.argtypes = [C.POINTER(pre_config), C.POINTER(vp)]
    lib.pre_destroy.argtypes = [vp]
    lib.pre_anticipate.argtypes = [vp, vp, vp, vp, vp, i64, vp, vp, vp]
    lib.pre_anticipate_static.argtypes = [C.c_int32, C.c_int32, vp, vp, vp, vp, i64, vp, vp, vp, vp]
    lib.pre_route_batch.argtypes = [vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.pre_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.pre_refine.argtypes = [vp] * 11
    lib.pre_tick.argtypes = [vp] * 10 + [C.c_double] * 3 + [vp] * 5
    lib.pre_route_admit.argtypes = [vp, vp, vp, i64, C.c_double, C.c_double, vp, vp, vp, i64] + [vp] * 12
    lib.pre_scaler_signals.argtypes = [vp, vp, C.c_double, C.c_double, C.c_double, vp, vp, vp, vp]
    lib.pre_ring_window.argtypes = [vp, vp, C.c_int32, vp, vp, vp]
    lib.pre_ring_fold.argtypes = [vp, vp, vp, vp, i64, vp, C.c_int32, vp, vp]
    lib.pre_ring_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, C.c_int32, vp, vp, vp, vp]
    lib.pre_ring_refine.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, C.c_int32, vp, vp, vp, vp]
    lib.pre_status.argtypes = [vp, vp]
    lib.pre_test_set_spin_limit.argtypes = [vp, C.c_uint32]
    lib.pre_route_select.argtypes = [vp, C.c_int32]
    lib.pre_last_cuda_error.argtypes = [vp]
    lib.pre_strerror.argtypes = [C.c_int]
    lib.pre_strerror.restype = C.c_char_p
    lib.pre_query.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.pre_query_layout.argtypes = [vp, C.POINTER(C.c_int64)]
    for name in EXPORTS:
        if name != "pre_strerror":
            getattr(lib, name).restype = C.c_int
    return lib


lib = _load()


class PreError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {pre_strerror(code)} ({code})")


def _ptr(t):
    """Device (or host) address of a tensor, None -> NULL, int passes through."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


def pre_strerror(code: int) -> str:
    return lib.pre_strerror(int(code)).decode()


def pre_create(n_instances, horizon, capacity_tokens, t_mem, beta, max_requests):
    """Returns (code, ctx handle or None)."""
    cfg = pre_config(int(n_instances), int(horizon), int(capacity_tokens), float(t_mem), float(beta),
                     int(max_requests))
    out = C.c_void_p()
    code = lib.pre_create(C.byref(cfg), C.byref(out))
    return code, (out.value if code == PRE_OK else None)


def pre_destroy(ctx):
    return lib.pre_destroy(ctx)


def pre_anticipate(ctx, prompt, generated, predicted, instance, n_requests, curves, current_d, stream=None):
    return lib.pre_anticipate(ctx, _ptr(prompt), _ptr(generated), _ptr(predicted), _ptr(instance),
                              int(n_requests), _ptr(curves), _ptr(current_d),
                              _stream() if stream is None else stream)


def pre_anticipate_static(n_instances, horizon, prompt, generated, predicted, instance, n_requests, curves,
                          current_d, flags=None, stream=None):
    """pre_anticipate for callers that must not allocate: no context, scratch built into the library."""
    return lib.pre_anticipate_static(int(n_instances), int(horizon), _ptr(prompt), _ptr(generated),
                                     _ptr(predicted), _ptr(instance), int(n_requests), _ptr(curves),
                                     _ptr(current_d), _ptr(flags), _stream() if stream is None else stream)


def pre_route_batch(ctx, arr_prompt, arr_predicted, n_arrivals, curves, queued_p, current_d, prompt, generated,
                    predicted, instance, n_requests, choice, score, stream=None):
    return lib.pre_route_batch(ctx, _ptr(arr_prompt), _ptr(arr_predicted), int(n_arrivals), _ptr(curves),
                               _ptr(queued_p), _ptr(current_d), _ptr(prompt), _ptr(generated), _ptr(predicted),
                               _ptr(instance), _ptr(n_requests), _ptr(choice), _ptr(score),
                               _stream() if stream is None else stream)


def pre_route_admit(ctx, arr_prompt, arr_predicted, n_arrivals, overload_level, overload_share, queue_prompt,
                    queue_predicted, queue_state, queue_capacity, queue_choice, curves, queued_p, current_d, prompt,
                    generated, predicted, instance, n_requests, choice, score, stream=None):
    return lib.pre_route_admit(ctx, _ptr(arr_prompt), _ptr(arr_predicted), int(n_arrivals), float(overload_level),
                               float(overload_share), _ptr(queue_prompt), _ptr(queue_predicted), _ptr(queue_state),
                               int(queue_capacity), _ptr(queue_choice), _ptr(curves), _ptr(queued_p),
                               _ptr(current_d), _ptr(prompt), _ptr(generated), _ptr(predicted), _ptr(instance),
                               _ptr(n_requests), _ptr(choice), _ptr(score), _stream() if stream is None else stream)


def pre_step(ctx, prompt, generated, predicted, instance, n_requests, curves, queued_p, current_d, stream=None):
    return lib.pre_step(ctx, _ptr(prompt), _ptr(generated), _ptr(predicted), _ptr(instance), _ptr(n_requests),
                        _ptr(curves), _ptr(queued_p), _ptr(current_d), _stream() if stream is None else stream)


def pre_refine(ctx, prompt, generated, predicted, instance, actual, n_requests, curves, current_d, counts,
               stream=None):
    return lib.pre_refine(ctx, _ptr(prompt), _ptr(generated), _ptr(predicted), _ptr(instance), _ptr(actual),
                          _ptr(n_requests), _ptr(curves), _ptr(current_d), _ptr(counts),
                          _stream() if stream is None else stream)


def pre_tick(ctx, prompt, generated, predicted, instance, actual, n_requests, curves, queued_p, current_d,
             overload_level, overload_share, idle_level, over_count, row_max, summary, counts, stream=None):
    return lib.pre_tick(ctx, _ptr(prompt), _ptr(generated), _ptr(predicted), _ptr(instance), _ptr(actual),
                        _ptr(n_requests), _ptr(curves), _ptr(queued_p), _ptr(current_d), float(overload_level),
                        float(overload_share), float(idle_level), _ptr(over_count), _ptr(row_max), _ptr(summary),
                        _ptr(counts), _stream() if stream is None else stream)


def pre_scaler_signals(ctx, curves, overload_level, overload_share, idle_level, over_count, row_max, summary,
                       stream=None):
    return lib.pre_scaler_signals(ctx, _ptr(curves), float(overload_level), float(overload_share),
                                  float(idle_level), _ptr(over_count), _ptr(row_max), _ptr(summary),
                                  _stream() if stream is None else stream)


def pre_ring_window(ctx, ring, width, head, window, stream=None):
    return lib.pre_ring_window(ctx, _ptr(ring), int(width), _ptr(head), _ptr(window),
                               _stream() if stream is None else stream)


def pre_ring_fold(ctx, arr_prompt, arr_predicted, choice, n_arrivals, ring, width, head, stream=None):
    return lib.pre_ring_fold(ctx, _ptr(arr_prompt), _ptr(arr_predicted), _ptr(choice), int(n_arrivals), _ptr(ring),
                             int(width), _ptr(head), _stream() if stream is None else stream)


def pre_ring_step(ctx, prompt, generated, predicted, instance, n_requests, ring, width, head, queued_p, current_d,
                  stream=None):
    return lib.pre_ring_step(ctx, _ptr(prompt), _ptr(generated), _ptr(predicted), _ptr(instance), _ptr(n_requests),
                             _ptr(ring), int(width), _ptr(head), _ptr(queued_p), _ptr(current_d),
                             _stream() if stream is None else stream)


def pre_ring_refine(ctx, prompt, generated, predicted, instance, actual, n_requests, ring, width, head, current_d,
                    counts, stream=None):
    return lib.pre_ring_refine(ctx, _ptr(prompt), _ptr(generated), _ptr(predicted), _ptr(instance), _ptr(actual),
                               _ptr(n_requests), _ptr(ring), int(width), _ptr(head), _ptr(current_d), _ptr(counts),
                               _stream() if stream is None else stream)


def pre_status(ctx, stream=None):
    return lib.pre_status(ctx, _stream() if stream is None else stream)


ROUTE_AUTO, ROUTE_SCAN, ROUTE_SUMMARY = 0, 1, 2


def pre_route_select(ctx, path):
    return lib.pre_route_select(ctx, int(path))


def pre_test_set_spin_limit(ctx, polls):
    return lib.pre_test_set_spin_limit(ctx, int(polls))


def pre_last_cuda_error(ctx):
    return lib.pre_last_cuda_error(ctx)


def pre_query(ctx):
    g, t = C.c_int32(), C.c_int32()
    code = lib.pre_query(ctx, C.byref(g), C.byref(t))
    return code, g.value, t.value


def pre_query_layout(ctx):
    out = (C.c_int64 * 4)()
    code = lib.pre_query_layout(ctx, out)
    return code, [int(v) for v in out]


def check(code: int, where: str = "preserve_b200"):
    if code != PRE_OK:
        raise PreError(code, where)
