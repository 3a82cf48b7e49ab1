"""Thin Python binding of the C ABI in include/fh.h (argument marshalling only).

Every step of the codec runs in the CUDA library; torch is used for device memory and streams.
There is no fallback: if the shared library is missing or no CUDA device is present the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfh_sm100a.so")

FH_OK, FH_ERR_ARG, FH_ERR_UNSUPPORTED, FH_ERR_CAPACITY, FH_ERR_NONFINITE, FH_ERR_CORRUPT, \
    FH_ERR_TIMEOUT, FH_ERR_CUDA = 0, -1, -2, -3, -4, -5, -6, -7
FH_F32, FH_BF16 = 0, 1
FH_SALIENT_AUTO, FH_SALIENT_OFF, FH_SALIENT_ALL, FH_SALIENT_CHANNEL, FH_SALIENT_TENSOR = 0, 1, 2, 3, 4
FH_KEEP, FH_COMPRESS, FH_EVICT = 0, 1, 2
FH_STATIC_MAX_PLANES = 131072
FH_DEBUG_WAIT_POLLS, FH_DEBUG_SILENT_TILE = 0, 1

EXPORTS = ["fh_default_params", "fh_version", "fh_device_count", "fh_compressed_bytes", "fh_compress",
           "fh_decompress", "fh_run_schedule", "fh_host_work_bytes", "fh_compress_host",
           "fh_decompress_host", "fh_compress_static", "fh_plan_generate", "fh_plan_measure", "fh_debug_set",
           "fh_kernel_launches",
           "fh_shutdown"]


class FhError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: fh_status {code}")
        self.code = code


class fh_tensor_desc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("n", C.c_int32), ("c", C.c_int32), ("h", C.c_int32),
                ("w", C.c_int32), ("tensor_id", C.c_uint64)]


class fh_params(C.Structure):
    _fields_ = [("bits", C.c_int32), ("salient_mode", C.c_int32), ("rho_num", C.c_int32),
                ("rho_den", C.c_int32), ("block", C.c_int32), ("tau_num", C.c_int32),
                ("tau_den", C.c_int32), ("eps", C.c_float), ("dense_bits", C.c_int32),
                ("rounding", C.c_int32), ("seed", C.c_uint64), ("entropy", C.c_int32), ("reserved", C.c_int32)]


class fh_sched_entry(C.Structure):
    _fields_ = [("desc", fh_tensor_desc), ("action", C.c_int32), ("d_dense", C.c_void_p),
                ("d_restored", C.c_void_p)]


class fh_sched_report(C.Structure):
    _fields_ = [("total_dense_bytes", C.c_uint64), ("total_packed_bytes", C.c_uint64),
                ("peak_packed_bytes", C.c_uint64), ("ms_forward", C.c_float), ("ms_backward", C.c_float),
                ("status", C.c_int32)]


class fh_plan_tensor(C.Structure):
    _fields_ = [("bytes", C.c_uint64), ("packed_bytes", C.c_uint64), ("t_compress", C.c_double),
                ("t_decompress", C.c_double), ("t_recompute", C.c_double)]


class fh_plan_op(C.Structure):
    _fields_ = [("time", C.c_double), ("inputs", C.POINTER(C.c_int32)), ("n_inputs", C.c_int32),
                ("outputs", C.POINTER(C.c_int32)), ("n_outputs", C.c_int32)]


class fh_plan_event(C.Structure):
    _fields_ = [("op", C.c_int32), ("tensor", C.c_int32), ("kind", C.c_int32)]


class fh_plan_report(C.Structure):
    _fields_ = [("peak_bytes", C.c_uint64), ("overhead_seconds", C.c_double), ("n_events", C.c_int32),
                ("n_over_budget", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2510_11400_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        D, P = C.POINTER(fh_tensor_desc), C.POINTER(fh_params)
        L.fh_default_params.argtypes = [P]
        L.fh_default_params.restype = None
        L.fh_version.restype = C.c_int
        L.fh_device_count.restype = C.c_int
        L.fh_compressed_bytes.argtypes = [D, P, C.c_int]
        L.fh_compressed_bytes.restype = C.c_size_t
        L.fh_compress.argtypes = [D, P, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.fh_compress.restype = C.c_int
        L.fh_decompress.argtypes = [C.c_void_p, C.c_size_t, D, C.c_void_p, C.c_void_p, C.c_void_p]
        L.fh_decompress.restype = C.c_int
        L.fh_run_schedule.argtypes = [C.POINTER(fh_sched_entry), C.c_int32, P, C.c_void_p, C.c_size_t,
                                      C.POINTER(fh_sched_report), C.c_void_p]
        L.fh_run_schedule.restype = C.c_int
        L.fh_host_work_bytes.argtypes = [D, P]
        L.fh_host_work_bytes.restype = C.c_size_t
        L.fh_compress_host.argtypes = [D, P, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p,
                                       C.c_size_t, C.c_void_p]
        L.fh_compress_host.restype = C.c_int
        L.fh_decompress_host.argtypes = [C.c_void_p, C.c_size_t, D, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_size_t, C.c_void_p]
        L.fh_decompress_host.restype = C.c_int
        L.fh_compress_static.argtypes = [D, P, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.fh_compress_static.restype = C.c_int
        L.fh_plan_generate.argtypes = [C.POINTER(fh_plan_op), C.c_int32, C.POINTER(fh_plan_tensor), C.c_int32, C.c_uint64,
                                       C.POINTER(C.c_int32), C.POINTER(fh_plan_event), C.c_int32,
                                       C.POINTER(fh_plan_report)]
        L.fh_plan_generate.restype = C.c_int
        L.fh_plan_measure.argtypes = [D, C.c_int32, P, C.POINTER(C.c_void_p), C.c_void_p, C.c_size_t, C.c_int32,
                                      C.POINTER(fh_plan_tensor), C.c_void_p]
        L.fh_plan_measure.restype = C.c_int
        L.fh_debug_set.argtypes = [C.c_int, C.c_uint64]
        L.fh_debug_set.restype = C.c_int
        L.fh_kernel_launches.restype = C.c_uint64
        L.fh_shutdown.restype = None
        _lib = L
    return _lib


def default_params(**kw) -> fh_params:
    p = fh_params()
    lib().fh_default_params(C.byref(p))
    for k, v in kw.items():
        if k == "rho":
            p.rho_num, p.rho_den = v
        elif k == "tau":
            p.tau_num, p.tau_den = v
        else:
            setattr(p, k, v)
    return p


def desc(shape: Sequence[int], dtype: int = FH_F32, tensor_id: int = 0) -> fh_tensor_desc:
    n, c, h, w = shape
    return fh_tensor_desc(dtype, n, c, h, w, tensor_id)


def compressed_bytes(d: fh_tensor_desc, p: fh_params, which: int = 0) -> int:
    return int(lib().fh_compressed_bytes(C.byref(d), C.byref(p), which))


def _stream_ptr(stream) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def fh_compress(d: fh_tensor_desc, p: fh_params, src, dst, out2=None, stream=None, capacity: Optional[int] = None) -> int:
    """Enqueue compression of the torch CUDA tensor `src` into the uint8 CUDA tensor `dst`.
    `out2` is an optional 2-element int64/uint64 CUDA tensor receiving (total bytes, status)."""
    cap = dst.numel() * dst.element_size() if capacity is None else capacity
    return int(lib().fh_compress(C.byref(d), C.byref(p), src.data_ptr(), dst.data_ptr(), cap,
                                 out2.data_ptr() if out2 is not None else None, _stream_ptr(stream)))


def fh_compress_static(d: fh_tensor_desc, p: fh_params, src, dst, out2=None, stream=None,
                       capacity: Optional[int] = None) -> int:
    """fh_compress for callers that must not allocate: same arguments and bytes, book-keeping scratch in a
    fixed array inside the library (at most FH_STATIC_MAX_PLANES planes; calls sharing a device must not
    overlap)."""
    cap = dst.numel() * dst.element_size() if capacity is None else capacity
    return int(lib().fh_compress_static(C.byref(d), C.byref(p), src.data_ptr(), dst.data_ptr(), cap,
                                        out2.data_ptr() if out2 is not None else None, _stream_ptr(stream)))


def fh_decompress(src, src_bytes: int, d: fh_tensor_desc, dst, status=None, stream=None) -> int:
    return int(lib().fh_decompress(src.data_ptr(), src_bytes, C.byref(d), dst.data_ptr(),
                                   status.data_ptr() if status is not None else None, _stream_ptr(stream)))


@dataclass
class SchedItem:
    desc: fh_tensor_desc
    action: int
    dense: object          # torch CUDA tensor
    restored: object       # torch CUDA tensor


def fh_run_schedule(items: List[SchedItem], p: fh_params, arena, stream=None) -> fh_sched_report:
    arr = (fh_sched_entry * len(items))()
    for i, it in enumerate(items):
        arr[i].desc = it.desc
        arr[i].action = it.action
        arr[i].d_dense = it.dense.data_ptr() if it.dense is not None else None
        arr[i].d_restored = it.restored.data_ptr() if it.restored is not None else None
    rep = fh_sched_report()
    rc = lib().fh_run_schedule(arr, len(items), C.byref(p), arena.data_ptr(),
                               arena.numel() * arena.element_size(), C.byref(rep), _stream_ptr(stream))
    if rc != FH_OK:
        raise FhError(rc, "fh_run_schedule")
    return rep


def host_work_bytes(d: fh_tensor_desc, p: Optional[fh_params]) -> int:
    return int(lib().fh_host_work_bytes(C.byref(d), C.byref(p) if p is not None else None))


def fh_compress_host(d: fh_tensor_desc, p: fh_params, h_src, h_dst, work, stream=None) -> Tuple[int, int]:
    """h_src / h_dst: CPU torch tensors (pinned for speed); work: uint8 CUDA tensor.  Returns
    (status, total bytes)."""
    out2 = (C.c_uint64 * 2)()
    rc = lib().fh_compress_host(C.byref(d), C.byref(p), h_src.data_ptr(), h_dst.data_ptr(),
                                h_dst.numel() * h_dst.element_size(), out2, work.data_ptr(),
                                work.numel() * work.element_size(), _stream_ptr(stream))
    return int(rc), int(out2[0])


def fh_decompress_host(h_src, src_bytes: int, d: fh_tensor_desc, h_dst, work, stream=None) -> int:
    st = C.c_uint64()
    rc = lib().fh_decompress_host(h_src.data_ptr(), src_bytes, C.byref(d), h_dst.data_ptr(), C.byref(st),
                                  work.data_ptr(), work.numel() * work.element_size(), _stream_ptr(stream))
    return int(rc)


def plan_generate(ops, tensors, memory_budget: int, max_events: int = 4096):
    """ops: [{time, inputs, outputs}], tensors: [{bytes, packed_bytes, t_compress, t_decompress, t_recompute}].
    Returns (status, actions, events, report)."""
    keep = []
    c_ops = (fh_plan_op * len(ops))()
    for i, op in enumerate(ops):
        ins = (C.c_int32 * len(op["inputs"]))(*op["inputs"])
        outs = (C.c_int32 * len(op["outputs"]))(*op["outputs"])
        keep += [ins, outs]
        c_ops[i] = fh_plan_op(op["time"], ins, len(op["inputs"]), outs, len(op["outputs"]))
    c_t = (fh_plan_tensor * len(tensors))(*[fh_plan_tensor(t["bytes"], t["packed_bytes"], t["t_compress"], t["t_decompress"],
                                                             t["t_recompute"]) for t in tensors])
    actions = (C.c_int32 * max(1, len(tensors)))()
    events = (fh_plan_event * max(1, max_events))()
    rep = fh_plan_report()
    rc = lib().fh_plan_generate(c_ops, len(ops), c_t, len(tensors), memory_budget, actions, events, max_events, C.byref(rep))
    n = min(rep.n_events, max_events)
    return int(rc), [int(a) for a in actions[:len(tensors)]], [(e.op, e.tensor, e.kind) for e in events[:n]], rep


def plan_measure(descs, p: fh_params, dense, work, repeats: int = 5, t_recompute=None, stream=None):
    """Measured costs of compression for plan generation: descs and dense are matching lists (descriptions, torch
    CUDA tensors); work is a uint8 CUDA tensor of at least host_work_bytes of the largest tensor.  Returns
    (status, list of dicts in the form plan_generate takes); t_recompute (list, seconds) is passed through."""
    n = len(descs)
    c_d = (fh_tensor_desc * n)(*descs)
    ptrs = (C.c_void_p * n)(*[t.data_ptr() for t in dense])
    out = (fh_plan_tensor * n)()
    for i in range(n):
        out[i].t_recompute = -1.0 if t_recompute is None else t_recompute[i]
    rc = lib().fh_plan_measure(c_d, n, C.byref(p), ptrs, work.data_ptr(), work.numel() * work.element_size(), repeats, out,
                               _stream_ptr(stream))
    return int(rc), [dict(bytes=int(o.bytes), packed_bytes=int(o.packed_bytes), t_compress=float(o.t_compress),
                          t_decompress=float(o.t_decompress), t_recompute=float(o.t_recompute)) for o in out]


def debug_set(what: int, value: int) -> int:
    """Host-side fault injection for the time-out test (see fh_debug_set in include/fh.h)."""
    return int(lib().fh_debug_set(what, value & 0xFFFFFFFFFFFFFFFF))


def kernel_launches() -> int:
    return int(lib().fh_kernel_launches())


def shutdown() -> None:
    if _lib is not None:
        _lib.fh_shutdown()


# ---- convenience for tests and the benchmark -------------------------------------------------

def compress_tensor(x, shape, dtype: int, p: fh_params, tensor_id: int = 0, capacity: Optional[int] = None):
    """Compress a flat CUDA tensor (float32, or int16/uint16/bfloat16 bit patterns for bf16).
    Synchronises.  Returns (status, packed uint8 CUDA tensor, total bytes)."""
    import torch
    d = desc(shape, dtype, tensor_id)
    cap = compressed_bytes(d, p, 1) if capacity is None else capacity
    dst = torch.empty(max(cap, 16), dtype=torch.uint8, device=x.device)
    out2 = torch.zeros(2, dtype=torch.int64, device=x.device)
    rc = fh_compress(d, p, x, dst, out2, capacity=cap)
    if rc != FH_OK:
        return rc, dst, 0
    torch.cuda.synchronize()
    total, st = (int(v) for v in out2.tolist())
    return st, dst, total


def decompress_tensor(packed, nbytes: int, shape, dtype: int):
    """Synchronises.  Returns (status, restored flat CUDA tensor)."""
    import torch
    d = desc(shape, dtype)
    n, c, h, w = shape
    out = torch.empty(n * c * h * w, dtype=torch.float32 if dtype == FH_F32 else torch.int16,
                      device=packed.device)
    st = torch.zeros(1, dtype=torch.int64, device=packed.device)
    rc = fh_decompress(packed, nbytes, d, out, st)
    if rc != FH_OK:
        return rc, out
    torch.cuda.synchronize()
    return int(st.item()), out
