"""Thin ctypes binding of the C-ABI library (include/tm_state.h): argument marshalling only.

Every function takes raw device addresses (ints, e.g. ``tensor.data_ptr()``) and a raw stream
handle (``torch.cuda.current_stream().cuda_stream``); every step of the path runs in the library's
kernels.  There is no CPU fallback: if ``libtm_state.so`` has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Iterable, List, Optional, Sequence, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtm_state.so")

TM_OK = 0
TM_ERR_ARG, TM_ERR_ALIGN, TM_ERR_CAPACITY, TM_ERR_OVERLAP = -1, -2, -3, -4
TM_ERR_RANK, TM_ERR_DTYPE, TM_ERR_CUDA, TM_ERR_TIMEOUT, TM_ERR_STATE = -5, -6, -7, -8, -9
TM_ERR_VERIFY, TM_ERR_TRANSPORT = -10, -11

_u64, _u32, _p, _int = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_int

# every symbol include/tm_state.h declares: name -> (restype, argtypes)
SIGNATURES = {
    "tm_options_get": (_int, [_p]),
    "tm_options_set": (_int, [_p]),
    "tm_plan_create": (_int, [_p, _u64, _u64, _p]),
    "tm_plan_create_range": (_int, [_p, _u64, _u64, _u64, _u64, _p]),
    "tm_plan_query": (_int, [_p, _p, _p, _p]),
    "tm_plan_range": (_int, [_p, _p, _p, _p, _p]),
    "tm_plan_emits": (_int, [_p, _p, _u64, _p]),
    "tm_shard_plan_create": (_int, [_p, _p, _u32, _u32, _u32, _p]),
    "tm_shard_plan_query": (_int, [_p, _p, _p]),
    "tm_shard_plan_bind": (_int, [_p, _p, _p, _p, _u64, _p]),
    "tm_shard_plan_extract": (_int, [_p, _p]),
    "tm_shard_plan_insert": (_int, [_p, _p]),
    "tm_shard_plan_status": (_int, [_p, _p, _p]),
    "tm_shard_plan_pieces": (_int, [_p, _p, _u64, _p, _p, _u64, _p, _p]),
    "tm_shard_plan_destroy": (None, [_p]),
    "tm_xfer_run_sender": (_int, [_u32, _u32, _u32, _p, _p]),
    "tm_xfer_run_receiver": (_int, [_u32, _u32, _u32, _p, _p]),
    "tm_xfer_create": (_int, [_p, _u64, _u64, _u64, _u32, _p]),
    "tm_xfer_query": (_int, [_p, _p, _p, _p, _p, _p]),
    "tm_xfer_bind": (_int, [_p, _p, _u64, _p, _u64, _p, _p, _p]),
    "tm_xfer_attach_shards": (_int, [_p, _p, _p, _u32, _u32, _u32, _p, _p, _p, _p, _u64, _p, _p]),
    "tm_xfer_send": (_int, [_p, _p, _p, _p, _u32, _p]),
    "tm_xfer_receive": (_int, [_p, _p, _p, _p, _u32, _p]),
    "tm_xfer_destroy": (None, [_p]),
    "tm_loopback_create": (_int, [_p, _p]),
    "tm_loopback_destroy": (None, [_p]),
    "tm_plan_offsets": (_int, [_p, _p]),
    "tm_plan_pieces": (_int, [_p, _p, _u64, _p, _p, _u64, _p]),
    "tm_plan_upload": (_int, [_p, _p, _u64, _p]),
    "tm_plan_status": (_int, [_p, _p, _p]),
    "tm_plan_destroy": (None, [_p]),
    "tm_state_pack": (_int, [_p, _p, _u64, _p, _p]),
    "tm_state_unpack": (_int, [_p, _p, _u64, _p]),
    "tm_state_unpack_verify": (_int, [_p, _p, _u64, _p, _p]),
    "tm_plan_attach_shards": (_int, [_p, _p, _p, _u32, _u32, _u32, _p, _p, _p, _p, _u64, _p, _p]),
    "tm_state_pack_emit": (_int, [_p, _p, _u64, _p, _p]),
    "tm_state_unpack_emit": (_int, [_p, _p, _u64, _p, _p]),
    "tm_shard_bounds": (_int, [_u64, _u32, _u32, _p, _p]),
    "tm_shard_workspace": (_int, [_p, _u64, _u32, _u32, _p]),
    "tm_shard_extract": (_int, [_p, _u64, _u32, _u32, _p, _u64, _p, _p, _u64, _p]),
    "tm_shard_extract_planes": (_int, [_p, _p, _u32, _u32, _u32, _p, _p, _p, _p, _u64, _p]),
    "tm_shard_insert": (_int, [_p, _u64, _u32, _u32, _p, _u64, _p, _p, _u64, _p]),
    "tm_shard_extract_static": (_int, [_p, _u64, _u32, _u32, _p, _u64, _p, _p]),
    "tm_selftest_bounded_wait": (_int, [_p, _u64, _p]),
    "tm_workspace_status": (_int, [_p, _p, _p]),
    "tm_checksum": (_int, [_p, _u64, _u64, _p, _p]),
    "tm_strerror": (ctypes.c_char_p, [_int]),
    "tm_last_cuda_error": (_int, []),
    "tm_launch_count": (_u64, []),
}


class TmDesc(ctypes.Structure):
    _fields_ = [("ptr", _p), ("nbytes", _u64), ("elem_size", _u32), ("plane", _u32)]


class TmOptions(ctypes.Structure):
    _fields_ = [("chunk_bytes", _u64), ("shard_chunk_bytes", _u64), ("small_bytes", _u64), ("group_bytes", _u64),
                ("cksum_tile_bytes", _u64), ("wait_limit_ns", _u64), ("group_max", _u32), ("ring_ctas_per_sm", _u32),
                ("ctas_per_sm", _u32), ("reserved", _u32)]


# callback types of tm_transport and tm_xfer_hooks
SEND_FN = ctypes.CFUNCTYPE(_int, _p, _u32, _p, _u64, _p, _u64, _p)
RECV_FN = ctypes.CFUNCTYPE(_int, _p, _u32, _p, _u64, _p, _u64, _p)
SEND_REPORT_FN = ctypes.CFUNCTYPE(_int, _p, ctypes.POINTER(_u32), _u32)
RECV_REPORT_FN = ctypes.CFUNCTYPE(_int, _p, ctypes.POINTER(_u32), _u32, ctypes.POINTER(_u32))
STEP_FN = ctypes.CFUNCTYPE(_int, _p, _u32, _u32)
BAD_WAVES_FN = ctypes.CFUNCTYPE(_int, _p, ctypes.POINTER(_u32), _u32, ctypes.POINTER(_u32), ctypes.POINTER(_u32))


class TmTransport(ctypes.Structure):
    _fields_ = [("ctx", _p), ("send", SEND_FN), ("recv", RECV_FN), ("send_report", SEND_REPORT_FN),
                ("recv_report", RECV_REPORT_FN)]


class TmXferHooks(ctypes.Structure):
    _fields_ = [("ctx", _p), ("pack", STEP_FN), ("send", STEP_FN), ("recv_report", RECV_REPORT_FN), ("recv", STEP_FN),
                ("unpack_verify", STEP_FN), ("bad_waves", BAD_WAVES_FN), ("send_report", SEND_REPORT_FN)]


class TmXferStats(ctypes.Structure):
    _fields_ = [("rounds", _u32), ("waves", _u32), ("waves_again", _u32), ("bad_buckets", _u32),
                ("first_bad_bucket", _u64), ("bytes", _u64)]

    def as_dict(self) -> dict:
        d = {name: getattr(self, name) for name, _ in self._fields_}
        if d["first_bad_bucket"] == (1 << 64) - 1:
            d["first_bad_bucket"] = None
        return d


class TmError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        super().__init__(f"{what}: {detail or status} (status {status})")
        self.status = status


_lib: Optional[ctypes.CDLL] = None


def load_library() -> ctypes.CDLL:
    """Loads libtm_state.so; raises if it is missing (build it with paper_2412_12636_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: the CUDA library has not been built "
                              "(run `python paper_2412_12636_b200/build.py`); there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(status: int, what: str) -> None:
    if status != TM_OK:
        L = load_library()
        detail = L.tm_strerror(status).decode()
        if status == TM_ERR_CUDA:
            detail += f" (cudaError {L.tm_last_cuda_error()})"
        raise TmError(status, what, detail)


def make_descs(descs: Iterable[Tuple[int, int, int, int]]):
    """ctypes array of tm_desc from (address, nbytes, elem_size, plane) tuples."""
    descs = list(descs)
    arr = (TmDesc * len(descs))()
    for i, (ptr, nbytes, elem_size, plane) in enumerate(descs):
        arr[i].ptr, arr[i].nbytes, arr[i].elem_size, arr[i].plane = ptr, nbytes, elem_size, plane
    return arr


def tm_options_get() -> dict:
    o = TmOptions()
    _check(load_library().tm_options_get(ctypes.byref(o)), "tm_options_get")
    return {name: getattr(o, name) for name, _ in TmOptions._fields_ if name != "reserved"}


def tm_options_set(**values) -> None:
    """Sets the named tuning values (the others keep their current value); no arguments restores the
    defaults.  Plans created afterwards use them."""
    L = load_library()
    if not values:
        _check(L.tm_options_set(None), "tm_options_set")
        return
    o = TmOptions()
    _check(L.tm_options_get(ctypes.byref(o)), "tm_options_get")
    for k, v in values.items():
        setattr(o, k, v)
    _check(L.tm_options_set(ctypes.byref(o)), "tm_options_set")


_PIECE_DTYPE = [("tensor", "<u8"), ("off", "<u8"), ("nbytes", "<u4"), ("pad", "<u4"), ("bucket", "<u4"), ("word0", "<u4")]


class Plan:
    """Owner of a tm_plan handle.  With `first_bucket` / `n_buckets` the plan covers that run of whole
    buckets of the stream only (tm_plan_create_range)."""

    def __init__(self, descs, bucket_bytes: int, first_bucket: Optional[int] = None, n_buckets: Optional[int] = None):
        L = load_library()
        self._h = _p()
        arr = descs if isinstance(descs, ctypes.Array) else make_descs(descs)
        if first_bucket is None:
            _check(L.tm_plan_create(arr, len(arr), bucket_bytes, ctypes.byref(self._h)), "tm_plan_create")
        else:
            _check(L.tm_plan_create_range(arr, len(arr), bucket_bytes, first_bucket, n_buckets, ctypes.byref(self._h)),
                   "tm_plan_create_range")
        self.n_desc = len(arr)
        t, n, w = _u64(), _u64(), _u64()
        _check(L.tm_plan_query(self._h, ctypes.byref(t), ctypes.byref(n), ctypes.byref(w)), "tm_plan_query")
        self.total_bytes, self.n_buckets, self.workspace_bytes = t.value, n.value, w.value
        f, b, wt, wn = _u64(), _u64(), _u64(), _u64()
        _check(L.tm_plan_range(self._h, ctypes.byref(f), ctypes.byref(b), ctypes.byref(wt), ctypes.byref(wn)), "tm_plan_range")
        self.first_bucket, self.stream_begin, self.whole_bytes, self.whole_buckets = f.value, b.value, wt.value, wn.value
        self.bucket_bytes = bucket_bytes

    def emits(self):
        """Emit records (numpy array with fields out, begin, len), one per piece; empty before attach."""
        import numpy as np
        L = load_library()
        n = _u64()
        _check(L.tm_plan_emits(self._h, None, 0, ctypes.byref(n)), "tm_plan_emits")
        out = np.zeros(n.value, dtype=np.dtype([("out", "<u8"), ("begin", "<u4"), ("len", "<u4")]))
        _check(L.tm_plan_emits(self._h, out.ctypes.data, out.size, None), "tm_plan_emits")
        return out

    def offsets(self) -> List[int]:
        out = (_u64 * self.n_desc)()
        _check(load_library().tm_plan_offsets(self._h, out), "tm_plan_offsets")
        return list(out)

    def pieces(self):
        """(pieces, item_first) of the work list as numpy arrays; pieces has fields tensor, off, nbytes,
        pad, bucket, word0."""
        import numpy as np
        L = load_library()
        np_, ni = _u64(), _u64()
        _check(L.tm_plan_pieces(self._h, None, 0, ctypes.byref(np_), None, 0, ctypes.byref(ni)), "tm_plan_pieces")
        pieces = np.zeros(np_.value, dtype=np.dtype(_PIECE_DTYPE))
        items = np.zeros(ni.value + 1, dtype=np.uint32)
        _check(L.tm_plan_pieces(self._h, pieces.ctypes.data, pieces.size, None, items.ctypes.data, items.size, None),
               "tm_plan_pieces")
        return pieces, items

    def upload(self, d_workspace: int, workspace_bytes: int, stream: int) -> None:
        _check(load_library().tm_plan_upload(self._h, d_workspace, workspace_bytes, stream), "tm_plan_upload")

    def status(self, stream: int) -> int:
        s = _int()
        _check(load_library().tm_plan_status(self._h, stream, ctypes.byref(s)), "tm_plan_status")
        return s.value

    @property
    def handle(self):
        return self._h

    def close(self) -> None:
        if self._h:
            load_library().tm_plan_destroy(self._h)
            self._h = _p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def tm_state_pack(plan: Plan, d_buckets: int, capacity: int, d_checksums: Optional[int], stream: int) -> None:
    _check(load_library().tm_state_pack(plan.handle, d_buckets, capacity, d_checksums, stream), "tm_state_pack")


def tm_state_unpack(plan: Plan, d_buckets: int, nbytes: int, stream: int) -> None:
    _check(load_library().tm_state_unpack(plan.handle, d_buckets, nbytes, stream), "tm_state_unpack")


def tm_state_unpack_verify(plan: Plan, d_buckets: int, nbytes: int, d_checksums: int, stream: int) -> None:
    _check(load_library().tm_state_unpack_verify(plan.handle, d_buckets, nbytes, d_checksums, stream),
           "tm_state_unpack_verify")


def tm_plan_attach_shards(plan: Plan, planes: Sequence[Tuple[int, int]], r: int, D: int,
                          d_outs: Optional[Sequence[int]], out_capacities: Optional[Sequence[int]],
                          d_workspace: Optional[int], workspace_bytes: int, stream: int) -> Tuple[List[int], int]:
    """`planes` = (first descriptor, count) per plane.  Returns (elements per shard, workspace bytes
    needed); with d_workspace None nothing is uploaded (size query)."""
    n = len(planes)
    first = (_u64 * n)(*[p[0] for p in planes])
    count = (_u64 * n)(*[p[1] for p in planes])
    outs = (_p * n)(*d_outs) if d_outs is not None else None
    caps = (_u64 * n)(*out_capacities) if out_capacities is not None else None
    got, need = (_u64 * n)(), _u64()
    _check(load_library().tm_plan_attach_shards(plan.handle, first, count, n, r, D, outs, caps, got, d_workspace,
                                                workspace_bytes, ctypes.byref(need), stream), "tm_plan_attach_shards")
    return list(got), need.value


def tm_state_pack_emit(plan: Plan, d_buckets: int, capacity: int, d_checksums: Optional[int], stream: int) -> None:
    _check(load_library().tm_state_pack_emit(plan.handle, d_buckets, capacity, d_checksums, stream),
           "tm_state_pack_emit")


def tm_state_unpack_emit(plan: Plan, d_buckets: int, nbytes: int, d_checksums: int, stream: int) -> None:
    _check(load_library().tm_state_unpack_emit(plan.handle, d_buckets, nbytes, d_checksums, stream),
           "tm_state_unpack_emit")


def tm_shard_bounds(n_elems: int, r: int, D: int) -> Tuple[int, int]:
    lo, hi = _u64(), _u64()
    _check(load_library().tm_shard_bounds(n_elems, r, D, ctypes.byref(lo), ctypes.byref(hi)), "tm_shard_bounds")
    return lo.value, hi.value


def tm_shard_workspace(descs, r: int, D: int) -> int:
    arr = descs if isinstance(descs, ctypes.Array) else make_descs(descs)
    w = _u64()
    _check(load_library().tm_shard_workspace(arr, len(arr), r, D, ctypes.byref(w)), "tm_shard_workspace")
    return w.value


def tm_shard_extract(descs, r: int, D: int, d_out: int, out_capacity: int, d_workspace: int,
                     workspace_bytes: int, stream: int) -> int:
    """Returns the number of elements written."""
    arr = descs if isinstance(descs, ctypes.Array) else make_descs(descs)
    n = _u64()
    _check(load_library().tm_shard_extract(arr, len(arr), r, D, d_out, out_capacity, ctypes.byref(n),
                                           d_workspace, workspace_bytes, stream), "tm_shard_extract")
    return n.value


def tm_shard_extract_planes(planes, r: int, D: int, d_outs: Sequence[int], out_capacities: Sequence[int],
                            d_workspace: int, workspace_bytes: int, stream: int) -> List[int]:
    """`planes` is a list of descriptor lists; returns the number of elements written per plane."""
    flat = [d for plane in planes for d in plane]
    arr = make_descs(flat)
    counts = (_u64 * len(planes))(*[len(p) for p in planes])
    outs = (_p * len(planes))(*d_outs)
    caps = (_u64 * len(planes))(*out_capacities)
    got = (_u64 * len(planes))()
    _check(load_library().tm_shard_extract_planes(arr, counts, len(planes), r, D, outs, caps, got, d_workspace,
                                                  workspace_bytes, stream), "tm_shard_extract_planes")
    return list(got)


def tm_shard_insert(descs, r: int, D: int, d_in: int, in_bytes: int, d_workspace: int, workspace_bytes: int,
                    stream: int) -> int:
    """Returns the number of elements written into the plane."""
    arr = descs if isinstance(descs, ctypes.Array) else make_descs(descs)
    n = _u64()
    _check(load_library().tm_shard_insert(arr, len(arr), r, D, d_in, in_bytes, ctypes.byref(n), d_workspace,
                                          workspace_bytes, stream), "tm_shard_insert")
    return n.value


class ShardPlan:
    """Owner of a tm_shard_plan handle: shard r of D of one or several planes, bound once to its flat
    buffers, then extract / insert are single launches."""

    def __init__(self, planes, r: int, D: int):
        L = load_library()
        self._h = _p()
        self.n_planes = len(planes)
        arr = make_descs([d for plane in planes for d in plane])
        counts = (_u64 * self.n_planes)(*[len(p) for p in planes])
        _check(L.tm_shard_plan_create(arr, counts, self.n_planes, r, D, ctypes.byref(self._h)), "tm_shard_plan_create")
        got, w = (_u64 * self.n_planes)(), _u64()
        _check(L.tm_shard_plan_query(self._h, got, ctypes.byref(w)), "tm_shard_plan_query")
        self.elems, self.workspace_bytes = list(got), w.value
        self.out_bytes = [n * plane[0][2] for n, plane in zip(self.elems, planes)]

    def bind(self, d_flats: Sequence[int], capacities: Sequence[int], d_workspace: int, workspace_bytes: int,
             stream: int) -> None:
        flats = (_p * self.n_planes)(*d_flats)
        caps = (_u64 * self.n_planes)(*capacities)
        _check(load_library().tm_shard_plan_bind(self._h, flats, caps, d_workspace, workspace_bytes, stream),
               "tm_shard_plan_bind")

    def extract(self, stream: int) -> None:
        _check(load_library().tm_shard_plan_extract(self._h, stream), "tm_shard_plan_extract")

    def insert(self, stream: int) -> None:
        _check(load_library().tm_shard_plan_insert(self._h, stream), "tm_shard_plan_insert")

    def status(self, stream: int) -> int:
        s = _int()
        _check(load_library().tm_shard_plan_status(self._h, stream, ctypes.byref(s)), "tm_shard_plan_status")
        return s.value

    def pieces(self):
        """(pieces, item_first, base): the bound work list; piece offsets are relative to `base`."""
        import numpy as np
        L = load_library()
        np_, ni, base = _u64(), _u64(), _u64()
        _check(L.tm_shard_plan_pieces(self._h, None, 0, ctypes.byref(np_), None, 0, ctypes.byref(ni), ctypes.byref(base)),
               "tm_shard_plan_pieces")
        pieces = np.zeros(np_.value, dtype=np.dtype(_PIECE_DTYPE))
        items = np.zeros(ni.value + 1, dtype=np.uint32)
        _check(L.tm_shard_plan_pieces(self._h, pieces.ctypes.data, pieces.size, None, items.ctypes.data, items.size,
                                      None, None), "tm_shard_plan_pieces")
        return pieces, items, base.value

    def close(self) -> None:
        if self._h:
            load_library().tm_shard_plan_destroy(self._h)
            self._h = _p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def tm_shard_extract_static(descs, r: int, D: int, d_out: int, out_capacity: int, stream: int) -> int:
    """Shard extract that uses the library's own fixed device scratch (no workspace argument, no
    device allocation); for callers that cannot allocate.  Returns the number of elements written."""
    arr = descs if isinstance(descs, ctypes.Array) else make_descs(descs)
    n = _u64()
    _check(load_library().tm_shard_extract_static(arr, len(arr), r, D, d_out, out_capacity, ctypes.byref(n),
                                                  stream), "tm_shard_extract_static")
    return n.value


def tm_selftest_bounded_wait(d_workspace: int, limit_ns: int, stream: int) -> None:
    _check(load_library().tm_selftest_bounded_wait(d_workspace, limit_ns, stream), "tm_selftest_bounded_wait")


def tm_workspace_status(d_workspace: int, stream: int) -> int:
    s = _int()
    _check(load_library().tm_workspace_status(d_workspace, stream, ctypes.byref(s)), "tm_workspace_status")
    return s.value


def tm_checksum(d_bytes: int, nbytes: int, bucket_bytes: int, d_checksums: int, stream: int) -> None:
    _check(load_library().tm_checksum(d_bytes, nbytes, bucket_bytes, d_checksums, stream), "tm_checksum")


def tm_launch_count() -> int:
    return load_library().tm_launch_count()
