"""ctypes binding of include/rstitch.h: same names, argument marshalling only.

PyTorch appears here for device memory and streams; nothing is computed in Python.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "librstitch.so")
_lib = None

TAU_NORMALIZED = 0x1
SAMPLE = 0x2
PATH_GEMV = 0x10
PATH_UMMA = 0x20

EXPORTS = [
    "rstitch_route", "rstitch_route_ex", "rstitch_route_host", "rstitch_create", "rstitch_destroy",
    "rstitch_workspace_bytes", "rstitch_compact", "rstitch_last_status", "rstitch_status_string",
    "rstitch_path_name", "rstitch_route_static", "rstitch_route_ex_host",
    "rstitch_alg1_init", "rstitch_alg1_plan", "rstitch_alg1_commit", "rstitch_router_forward",
    "rstitch_router_route", "rstitch_router_route_alg1", "rstitch_probe_read_stream",
]


class RstitchError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %d (%s)" % (where, status, status_string(status)))


class _Args(C.Structure):
    _fields_ = [
        ("hidden", C.c_void_p), ("W_head", C.c_void_p),
        ("R", C.c_int32), ("B", C.c_int32), ("d", C.c_int32), ("V", C.c_int32), ("n_src", C.c_int32),
        ("tau", C.c_float), ("flags", C.c_uint32),
        ("row_idx", C.c_void_p), ("row_seq", C.c_void_p), ("n_rows_dev", C.c_void_p),
        ("seq_len", C.c_void_p), ("kv_len", C.c_void_p),
        ("tok_out", C.c_void_p), ("ent_out", C.c_void_p), ("route_mask", C.c_void_p),
        ("llm_idx", C.c_void_p), ("llm_count", C.c_void_p),
        ("llm_span", C.c_void_p), ("llm_row_off", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("temperature", C.c_float), ("seed", C.c_uint64), ("draw", C.c_uint64),
        ("alg1_tail", C.c_void_p),
    ]


class DevStat(C.Structure):
    _fields_ = [("nan_rows", C.c_uint32), ("bad_row_idx", C.c_uint32), ("bad_span", C.c_uint32),
                ("timeouts", C.c_uint32), ("timeout_site", C.c_uint32), ("launches", C.c_uint32),
                ("reserved", C.c_uint32 * 2)]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k in
                ("nan_rows", "bad_row_idx", "bad_span", "timeouts", "timeout_site", "launches")}


class LatencyModel(C.Structure):
    """rstitch_latency_model_t: Eq. 5 coefficients (a, b, c, d), milliseconds."""
    _fields_ = [("a", C.c_double), ("b", C.c_double), ("c", C.c_double), ("d", C.c_double)]


ROUTER_KEYS = ("W_in", "b_in", "W1", "b1", "W2", "b2", "ln_g", "ln_b", "W_out", "b_out")


class _Router(C.Structure):
    _fields_ = [("d", C.c_int32), ("h", C.c_int32), ("ff", C.c_int32), ("n_blocks", C.c_int32)] + \
               [(k, C.c_void_p) for k in ROUTER_KEYS]


class _Alg1State(C.Structure):
    _fields_ = [("active", C.c_void_p), ("kv_slm", C.c_void_p), ("kv_llm", C.c_void_p), ("seq_len", C.c_void_p),
                ("n_out", C.c_void_p), ("done", C.c_void_p), ("iters", C.c_void_p), ("kept", C.c_void_p),
                ("steps", C.c_void_p), ("lat_ms", C.c_void_p), ("y", C.c_void_p), ("y_cap", C.c_int32)]


class _Alg1Tail(C.Structure):
    _fields_ = [("state", C.c_void_p), ("n_seq", C.c_int32), ("model", C.c_int32),
                ("run_idx", C.c_void_p), ("run_count", C.c_void_p), ("row_off", C.c_void_p),
                ("eos_id", C.c_int32), ("plan_next", C.c_int32), ("t_max", C.c_int32),
                ("latency", LatencyModel * 2),
                ("next_run_idx", C.c_void_p * 2), ("next_run_count", C.c_void_p * 2), ("next_n_inf", C.c_void_p * 2),
                ("next_n_kv", C.c_void_p * 2), ("next_row_off", C.c_void_p * 2)]


def library_path() -> str:
    return _LIB_PATH


def lib():
    """The loaded C library.  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                "librstitch.so is missing (%s): build it with "
                "`python -m paper_2507_17307_b200.build`; there is no fallback path" % _LIB_PATH)
        L = C.CDLL(_LIB_PATH)
        vp, i, f = C.c_void_p, C.c_int, C.c_float
        L.rstitch_route.argtypes = [vp, vp, i, i, i, f, vp, vp, vp, vp, vp]
        L.rstitch_route.restype = i
        L.rstitch_route_ex.argtypes = [vp, C.POINTER(_Args), vp]
        L.rstitch_route_ex.restype = i
        L.rstitch_route_ex_host.argtypes = [vp, C.POINTER(_Args), vp]
        L.rstitch_route_ex_host.restype = i
        L.rstitch_route_host.argtypes = [vp, vp, vp, i, i, i, f, vp, vp, vp, vp, vp, vp]
        L.rstitch_route_host.restype = i
        L.rstitch_create.argtypes = [C.POINTER(vp), i, i, i]
        L.rstitch_create.restype = i
        L.rstitch_destroy.argtypes = [vp]
        L.rstitch_destroy.restype = i
        L.rstitch_workspace_bytes.argtypes = [i, i, i]
        L.rstitch_workspace_bytes.restype = C.c_size_t
        L.rstitch_compact.argtypes = [vp, i, vp, vp, vp]
        L.rstitch_compact.restype = i
        L.rstitch_last_status.argtypes = [vp, C.POINTER(DevStat)]
        L.rstitch_last_status.restype = i
        L.rstitch_status_string.argtypes = [i]
        L.rstitch_status_string.restype = C.c_char_p
        L.rstitch_path_name.argtypes = [i, i, i, C.c_uint32]
        L.rstitch_path_name.restype = C.c_char_p
        L.rstitch_route_static.argtypes = [vp, vp, i, i, i, f, vp, vp, vp, vp, vp, vp]
        L.rstitch_route_static.restype = i
        L.rstitch_probe_read_stream.argtypes = [vp, C.c_size_t, vp, vp]
        L.rstitch_probe_read_stream.restype = i
        L.rstitch_selftest_wait.argtypes = [vp, vp]
        L.rstitch_selftest_wait.restype = i
        L.rstitch_shard_stats.argtypes = [vp, C.POINTER(_Args), C.c_int32, vp, vp]
        L.rstitch_shard_stats.restype = i
        L.rstitch_shard_route.argtypes = [vp, C.POINTER(_Args), vp, C.c_int32, vp]
        L.rstitch_shard_route.restype = i
        L.rstitch_router_forward.argtypes = [C.POINTER(_Router), vp, i, vp, vp, i, vp, vp, vp, vp]
        L.rstitch_router_forward.restype = i
        L.rstitch_router_route.argtypes = [C.POINTER(_Router), vp, i, vp, vp, i, vp, vp, vp, vp, vp, vp]
        L.rstitch_router_route.restype = i
        L.rstitch_router_route_alg1.argtypes = [C.POINTER(_Router), vp, i, vp, vp, vp, i, vp, vp, vp, vp, vp, vp,
                                                C.POINTER(_Alg1Tail), vp]
        L.rstitch_router_route_alg1.restype = i
        L.rstitch_alg1_init.argtypes = [C.POINTER(_Alg1State), i, vp, vp]
        L.rstitch_alg1_init.restype = i
        L.rstitch_alg1_plan.argtypes = [C.POINTER(_Alg1State), i, i, i, C.POINTER(LatencyModel), vp, vp, vp, vp, vp, vp]
        L.rstitch_alg1_plan.restype = i
        L.rstitch_alg1_commit.argtypes = [C.POINTER(_Alg1State), i, i, vp, vp, vp, vp, vp, C.c_int32, vp]
        L.rstitch_alg1_commit.restype = i
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().rstitch_status_string(int(status)).decode()


def path_name(R: int, d: int, V: int, flags: int = 0) -> str:
    return lib().rstitch_path_name(int(R), int(d), int(V), int(flags)).decode()


def workspace_bytes(R: int, d: int, V: int) -> int:
    return int(lib().rstitch_workspace_bytes(int(R), int(d), int(V)))


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _stream_ptr(stream) -> Optional[int]:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) or None


class Handle:
    """rstitch_create / rstitch_destroy."""

    def __init__(self, maxR: int, max_d: int, maxV: int):
        h = C.c_void_p()
        st = lib().rstitch_create(C.byref(h), int(maxR), int(max_d), int(maxV))
        if st != 0:
            raise RstitchError(st, "rstitch_create")
        self._h = h

    @property
    def ptr(self):
        return self._h

    def destroy(self):
        if self._h is not None and self._h.value:
            lib().rstitch_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


@dataclass
class RouteOutputs:
    """Device buffers one call writes."""
    tok: "object"
    ent: "object"
    mask: "object"
    llm_idx: "object"
    llm_count: "object"
    llm_span: "object" = None
    llm_row_off: "object" = None

    @staticmethod
    def allocate(R: int, B: int, device, spans: bool = False) -> "RouteOutputs":
        import torch
        o = RouteOutputs(
            tok=torch.full((max(R, 1),), -1, dtype=torch.int32, device=device),
            ent=torch.full((max(R, 1),), -1.0, dtype=torch.float32, device=device),
            mask=torch.full((max(B, 1),), 255, dtype=torch.uint8, device=device),
            llm_idx=torch.full((max(B, 1),), -1, dtype=torch.int32, device=device),
            llm_count=torch.full((1,), -1, dtype=torch.int32, device=device))
        if spans:
            o.llm_span = torch.full((max(B, 1),), -1, dtype=torch.int32, device=device)
            o.llm_row_off = torch.full((B + 1,), -1, dtype=torch.int32, device=device)
        return o


def route(hidden, W_head, tau: float, out: Optional[RouteOutputs] = None) -> RouteOutputs:
    """rstitch_route: B rows, one decision per row, on the legacy default stream."""
    B, d = int(hidden.shape[0]), int(hidden.shape[1])
    V = int(W_head.shape[0])
    if out is None:
        out = RouteOutputs.allocate(B, B, hidden.device)
    st = lib().rstitch_route(_ptr(hidden), _ptr(W_head), B, d, V, float(tau), _ptr(out.tok), _ptr(out.ent),
                             _ptr(out.mask), _ptr(out.llm_idx), _ptr(out.llm_count))
    if st != 0:
        raise RstitchError(st, "rstitch_route")
    return out


def route_ex(handle: Handle, hidden, W_head, tau: float, *, R: Optional[int] = None,
             B: Optional[int] = None, row_idx=None, row_seq=None, n_rows_dev=None, seq_len=None,
             kv_len=None, flags: int = 0, stream=None, out: Optional[RouteOutputs] = None,
             workspace=None, check: bool = True, sample=None, alg1_tail=None):
    """rstitch_route_ex.  Returns the outputs (or the status when check=False).
    sample = (temperature, seed, draw) asks for a sampled token (RSTITCH_SAMPLE);
    alg1_tail = Alg1State.tail(...) lets the call run Algorithm 1's decision block itself."""
    n_src, d = int(hidden.shape[0]), int(hidden.shape[1])
    V = int(W_head.shape[0])
    if R is None:
        R = int(row_idx.shape[0]) if row_idx is not None else n_src
    if B is None:
        B = R
    if out is None:
        out = RouteOutputs.allocate(R, B, hidden.device, spans=seq_len is not None)
    a = _Args()
    a.hidden, a.W_head = _ptr(hidden), _ptr(W_head)
    a.R, a.B, a.d, a.V, a.n_src = R, B, d, V, n_src
    a.tau, a.flags = float(tau), int(flags)
    a.row_idx, a.row_seq, a.n_rows_dev = _ptr(row_idx), _ptr(row_seq), _ptr(n_rows_dev)
    a.seq_len, a.kv_len = _ptr(seq_len), _ptr(kv_len)
    a.tok_out, a.ent_out, a.route_mask = _ptr(out.tok), _ptr(out.ent), _ptr(out.mask)
    a.llm_idx, a.llm_count = _ptr(out.llm_idx), _ptr(out.llm_count)
    a.llm_span, a.llm_row_off = _ptr(out.llm_span), _ptr(out.llm_row_off)
    if workspace is not None:
        a.workspace, a.workspace_bytes = _ptr(workspace), int(workspace.numel() * workspace.element_size())
    if sample is not None:
        a.flags |= SAMPLE
        a.temperature, a.seed, a.draw = float(sample[0]), int(sample[1]), int(sample[2])
    if alg1_tail is not None:
        a.alg1_tail = C.addressof(alg1_tail)
    st = lib().rstitch_route_ex(handle.ptr, C.byref(a), _stream_ptr(stream))
    if not check:
        return st
    if st != 0:
        raise RstitchError(st, "rstitch_route_ex")
    return out


SHARD_WORDS = 5


def shard_stats(handle: Handle, hidden, W_shard, v_base: int, *, R: Optional[int] = None, row_idx=None,
                n_rows_dev=None, flags: int = 0, stream=None, out=None, sample=None, check: bool = True):
    """rstitch_shard_stats: the head on one vocabulary shard (rows [v_base, v_base + len(W_shard)) of the
    whole W_head).  Returns the int32 tensor [R, SHARD_WORDS] of per-row statistics (float words viewed
    as int32 so that a gather moves them bit for bit)."""
    import torch
    n_src, d = int(hidden.shape[0]), int(hidden.shape[1])
    if R is None:
        R = int(row_idx.shape[0]) if row_idx is not None else n_src
    if out is None:
        out = torch.zeros((R, SHARD_WORDS), dtype=torch.int32, device=hidden.device)
    a = _Args()
    a.hidden, a.W_head = _ptr(hidden), _ptr(W_shard)
    a.R, a.B, a.d, a.V, a.n_src = R, R, d, int(W_shard.shape[0]), n_src
    a.flags = int(flags)
    a.row_idx, a.n_rows_dev = _ptr(row_idx), _ptr(n_rows_dev)
    if sample is not None:
        a.flags |= SAMPLE
        a.temperature, a.seed, a.draw = float(sample[0]), int(sample[1]), int(sample[2])
    st = lib().rstitch_shard_stats(handle.ptr, C.byref(a), int(v_base), _ptr(out), _stream_ptr(stream))
    if not check:
        return st
    if st != 0:
        raise RstitchError(st, "rstitch_shard_stats")
    return out


def shard_route(handle: Handle, gathered, V: int, tau: float, *, R: Optional[int] = None, B: Optional[int] = None,
                row_seq=None, n_rows_dev=None, seq_len=None, kv_len=None, flags: int = 0, stream=None,
                out: Optional[RouteOutputs] = None, check: bool = True):
    """rstitch_shard_route: merge of the gathered shards [n_shards, R, SHARD_WORDS] and the routing tail;
    V is the size of the whole vocabulary."""
    n_shards = int(gathered.shape[0])
    if R is None:
        R = int(gathered.shape[1])
    if B is None:
        B = R
    if out is None:
        out = RouteOutputs.allocate(R, B, gathered.device, spans=seq_len is not None)
    a = _Args()
    a.R, a.B, a.V = R, B, int(V)
    a.tau, a.flags = float(tau), int(flags)
    a.row_seq, a.n_rows_dev = _ptr(row_seq), _ptr(n_rows_dev)
    a.seq_len, a.kv_len = _ptr(seq_len), _ptr(kv_len)
    a.tok_out, a.ent_out, a.route_mask = _ptr(out.tok), _ptr(out.ent), _ptr(out.mask)
    a.llm_idx, a.llm_count = _ptr(out.llm_idx), _ptr(out.llm_count)
    a.llm_span, a.llm_row_off = _ptr(out.llm_span), _ptr(out.llm_row_off)
    st = lib().rstitch_shard_route(handle.ptr, C.byref(a), _ptr(gathered), n_shards, _stream_ptr(stream))
    if not check:
        return st
    if st != 0:
        raise RstitchError(st, "rstitch_shard_route")
    return out


STATIC_MAX_ROWS = 16


def route_static(hidden, W_head, tau: float, out: RouteOutputs, stream=None, check: bool = True):
    """rstitch_route_static: the allocation-free variant (scratch inside the library image).

    For callers that may not allocate device memory, so `out` must be given: this wrapper creates
    no tensor.  At most STATIC_MAX_ROWS rows; calls sharing a device must not overlap on the GPU.
    """
    B, d = int(hidden.shape[0]), int(hidden.shape[1])
    st = lib().rstitch_route_static(_ptr(hidden), _ptr(W_head), B, d, int(W_head.shape[0]), float(tau),
                                    _ptr(out.tok), _ptr(out.ent), _ptr(out.mask), _ptr(out.llm_idx),
                                    _ptr(out.llm_count), _stream_ptr(stream))
    if check and st != 0:
        raise RstitchError(st, "rstitch_route_static")
    return out if check else st


class PreparedCall:
    """A filled rstitch_args_t kept alive with its tensors, so that a step loop pays one C call
    per step and no Python marshalling.  launch() is rstitch_route_ex with those arguments."""

    def __init__(self, handle: Handle, hidden, W_head, tau: float, out: RouteOutputs, *, R=None, B=None,
                 row_idx=None, row_seq=None, n_rows_dev=None, seq_len=None, kv_len=None, flags=0,
                 stream=None, alg1_tail=None):
        n_src, d = int(hidden.shape[0]), int(hidden.shape[1])
        if R is None:
            R = int(row_idx.shape[0]) if row_idx is not None else n_src
        if B is None:
            B = R
        a = _Args()
        a.hidden, a.W_head = _ptr(hidden), _ptr(W_head)
        a.R, a.B, a.d, a.V, a.n_src = R, B, d, int(W_head.shape[0]), n_src
        a.tau, a.flags = float(tau), int(flags)
        a.row_idx, a.row_seq, a.n_rows_dev = _ptr(row_idx), _ptr(row_seq), _ptr(n_rows_dev)
        a.seq_len, a.kv_len = _ptr(seq_len), _ptr(kv_len)
        a.tok_out, a.ent_out, a.route_mask = _ptr(out.tok), _ptr(out.ent), _ptr(out.mask)
        a.llm_idx, a.llm_count = _ptr(out.llm_idx), _ptr(out.llm_count)
        a.llm_span, a.llm_row_off = _ptr(out.llm_span), _ptr(out.llm_row_off)
        if alg1_tail is not None:
            a.alg1_tail = C.addressof(alg1_tail)
        self._keep = (handle, hidden, W_head, out, row_idx, row_seq, n_rows_dev, seq_len, kv_len, alg1_tail)
        self._args = a
        self._ref = C.byref(a)
        self._h = handle.ptr
        self._stream = _stream_ptr(stream)
        self._fn = lib().rstitch_route_ex
        self.out = out

    def launch(self) -> int:
        return self._fn(self._h, self._ref, self._stream)


def route_host(handle: Handle, hidden_host, W_head_dev, tau: float, host_out: dict, stream=None):
    """rstitch_route_host: per-step data in host buffers (torch CPU tensors, ideally pinned).

    host_out holds CPU tensors 'tok' int32 [B], 'ent' float32 [B], 'mask' uint8 [B],
    'llm_idx' int32 [B], 'llm_count' int32 [1]; returns after the stream is synchronised.
    """
    B, d = int(hidden_host.shape[0]), int(hidden_host.shape[1])
    V = int(W_head_dev.shape[0])
    st = lib().rstitch_route_host(handle.ptr, _ptr(hidden_host), _ptr(W_head_dev), B, d, V, float(tau),
                                  _ptr(host_out["tok"]), _ptr(host_out["ent"]), _ptr(host_out["mask"]),
                                  _ptr(host_out["llm_idx"]), _ptr(host_out["llm_count"]),
                                  _stream_ptr(stream))
    if st != 0:
        raise RstitchError(st, "rstitch_route_host")
    return host_out


class PreparedHostCall:
    """rstitch_route_ex_host with its rstitch_args_t filled once: hidden, the optional index arrays
    and every output are CPU tensors (ideally pinned), W_head a device tensor.  host_out holds 'tok'
    int32 [R], 'ent' float32 [R], 'mask' uint8 [B], 'llm_idx' int32 [B], 'llm_count' int32 [1] and,
    with seq_len / kv_len, 'llm_span' int32 [B] and 'llm_row_off' int32 [B + 1]."""

    def __init__(self, handle: Handle, hidden_host, W_head_dev, tau: float, host_out: dict, *, R=None, B=None,
                 row_idx=None, row_seq=None, seq_len=None, kv_len=None, flags=0, stream=None):
        n_src, d = int(hidden_host.shape[0]), int(hidden_host.shape[1])
        if R is None:
            R = int(row_idx.shape[0]) if row_idx is not None else n_src
        if B is None:
            B = R
        a = _Args()
        a.hidden, a.W_head = _ptr(hidden_host), _ptr(W_head_dev)
        a.R, a.B, a.d, a.V, a.n_src = R, B, d, int(W_head_dev.shape[0]), n_src
        a.tau, a.flags = float(tau), int(flags)
        a.row_idx, a.row_seq = _ptr(row_idx), _ptr(row_seq)
        a.seq_len, a.kv_len = _ptr(seq_len), _ptr(kv_len)
        a.tok_out, a.ent_out, a.route_mask = _ptr(host_out["tok"]), _ptr(host_out["ent"]), _ptr(host_out["mask"])
        a.llm_idx, a.llm_count = _ptr(host_out["llm_idx"]), _ptr(host_out["llm_count"])
        a.llm_span, a.llm_row_off = _ptr(host_out.get("llm_span")), _ptr(host_out.get("llm_row_off"))
        self._keep = (handle, hidden_host, W_head_dev, host_out, row_idx, row_seq, seq_len, kv_len)
        self.args = a
        self._ref = C.byref(a)
        self._h = handle.ptr
        self._stream = _stream_ptr(stream)
        self._fn = lib().rstitch_route_ex_host
        self.out = host_out

    def set_rows(self, R: int, B: Optional[int] = None):
        """Change the row count between steps (e.g. to the llm_count an earlier call returned)."""
        self.args.R = int(R)
        self.args.B = int(R if B is None else B)

    def launch(self) -> int:
        return self._fn(self._h, self._ref, self._stream)


def route_ex_host(handle: Handle, hidden_host, W_head_dev, tau: float, host_out: dict, **kw):
    """rstitch_route_ex_host, one call; see PreparedHostCall for the arguments."""
    st = PreparedHostCall(handle, hidden_host, W_head_dev, tau, host_out, **kw).launch()
    if st != 0:
        raise RstitchError(st, "rstitch_route_ex_host")
    return host_out


def compact(mask, idx=None, count=None, stream=None):
    """rstitch_compact: (llm_idx int32 [B], llm_count int32 [1]) of a uint8 device mask."""
    import torch
    B = int(mask.shape[0])
    if idx is None:
        idx = torch.full((max(B, 1),), -1, dtype=torch.int32, device=mask.device)
    if count is None:
        count = torch.full((1,), -1, dtype=torch.int32, device=mask.device)
    st = lib().rstitch_compact(_ptr(mask), B, _ptr(idx), _ptr(count), _stream_ptr(stream))
    if st != 0:
        raise RstitchError(st, "rstitch_compact")
    return idx, count


SELFTEST_SITE = 0x7E57


def probe_read_stream(buf, gave_up, stream=None) -> int:
    """One read-only pass over a device buffer (measurement aid); gave_up: zeroed uint32/int32 tensor [1]."""
    st = lib().rstitch_probe_read_stream(_ptr(buf), buf.numel() * buf.element_size(), _ptr(gave_up),
                                         _stream_ptr(stream))
    if st != 0:
        raise RstitchError(st, "rstitch_probe_read_stream")
    return st


def selftest_wait(handle: Handle, stream=None) -> int:
    """rstitch_selftest_wait: makes one bounded device-side wait run out (about a millisecond); the next
    last_status(handle) reports the timeout."""
    return lib().rstitch_selftest_wait(handle.ptr, _stream_ptr(stream))


def last_status(handle: Optional[Handle] = None) -> dict:
    """rstitch_last_status: device status word as a dict (adds 'status')."""
    s = DevStat()
    st = lib().rstitch_last_status(handle.ptr if handle is not None else None, C.byref(s))
    if st not in (0, -6):
        raise RstitchError(st, "rstitch_last_status")
    out = s.as_dict()
    out["status"] = st
    return out


class Alg1State:
    """rstitch_alg1_state_t with its device arrays (torch tensors), plus the per-round run lists."""

    INT_FIELDS = ("active", "kv_slm", "kv_llm", "seq_len", "n_out", "done", "iters")

    def __init__(self, B: int, y_cap: int, device="cuda"):
        import torch
        self.B, self.y_cap = int(B), int(y_cap)
        n = max(self.B, 1)
        for k in self.INT_FIELDS:
            setattr(self, k, torch.zeros(n, dtype=torch.int32, device=device))
        self.kept = torch.zeros(2 * n, dtype=torch.int32, device=device)
        self.steps = torch.zeros(2 * n, dtype=torch.int32, device=device)
        self.lat_ms = torch.zeros(n, dtype=torch.float64, device=device)
        self.y = torch.full((n, self.y_cap), -1, dtype=torch.int32, device=device)
        # run lists of the two plan calls of a round, one set per model (both plans come before
        # either commit: a sequence handed over by a commit must not run again in the same round)
        mk = lambda shape, fill=0: torch.full(shape, fill, dtype=torch.int32, device=device)
        self.run_idx = [mk((n,), -1), mk((n,), -1)]
        self.run_count = [mk((1,)), mk((1,))]
        self.n_inf = [mk((n,)), mk((n,))]
        self.n_kv = [mk((n,)), mk((n,))]
        self.row_off = [mk((n + 1,)), mk((n + 1,))]
        c = _Alg1State()
        for k in self.INT_FIELDS + ("kept", "steps", "lat_ms", "y"):
            setattr(c, k, _ptr(getattr(self, k)))
        c.y_cap = self.y_cap
        self._c = c

    def init(self, prompt_len, stream=None):
        st = lib().rstitch_alg1_init(C.byref(self._c), self.B, _ptr(prompt_len), _stream_ptr(stream))
        if st != 0:
            raise RstitchError(st, "rstitch_alg1_init")

    def plan(self, model: int, t_max: int, latency: LatencyModel, stream=None):
        st = lib().rstitch_alg1_plan(C.byref(self._c), self.B, int(model), int(t_max), C.byref(latency),
                                     _ptr(self.run_idx[model]), _ptr(self.run_count[model]), _ptr(self.n_inf[model]),
                                     _ptr(self.n_kv[model]), _ptr(self.row_off[model]), _stream_ptr(stream))
        if st != 0:
            raise RstitchError(st, "rstitch_alg1_plan")

    def tail(self, model: int, eos_id: int, spans: bool = True, plan_next: bool = False, t_max: int = 0,
             latency=None):
        """rstitch_alg1_tail_t for a routing call on `model`'s batch (pass it as alg1_tail=): the call
        then applies the decision block to plan(model)'s run list itself and, with plan_next, plans the
        next round for both models (latency = the two models' LatencyModel) into this object's run lists.
        Keep the returned structure alive while calls that use it may still be issued."""
        t = _Alg1Tail()
        t.state = C.addressof(self._c)
        t.n_seq, t.model, t.eos_id = self.B, int(model), int(eos_id)
        t.run_idx, t.run_count = _ptr(self.run_idx[model]), _ptr(self.run_count[model])
        t.row_off = _ptr(self.row_off[model]) if spans else None
        t.plan_next, t.t_max = int(bool(plan_next)), int(t_max)
        if plan_next:
            for m in (0, 1):
                t.latency[m] = latency[m]
                t.next_run_idx[m], t.next_run_count[m] = _ptr(self.run_idx[m]), _ptr(self.run_count[m])
                t.next_n_inf[m], t.next_n_kv[m] = _ptr(self.n_inf[m]), _ptr(self.n_kv[m])
                t.next_row_off[m] = _ptr(self.row_off[m])
        t._keep = self
        return t

    def commit(self, model: int, tok, mask, eos_id: int, spans: bool = True, stream=None):
        """Applies the decision block to the run list of plan(model).  spans=True: tok has one entry
        per row of the model's batch and a sequence's token is the last row of its span; spans=False:
        tok has one entry per run entry."""
        st = lib().rstitch_alg1_commit(C.byref(self._c), self.B, int(model), _ptr(self.run_idx[model]),
                                       _ptr(self.run_count[model]), _ptr(self.row_off[model]) if spans else None,
                                       _ptr(tok), _ptr(mask), int(eos_id), _stream_ptr(stream))
        if st != 0:
            raise RstitchError(st, "rstitch_alg1_commit")


class Router:
    """rstitch_router_t over device tensors (float32): the R-Stitch+ router's weights."""

    def __init__(self, weights: dict):
        self.w = weights
        h, d = weights["W_in"].shape
        L, ff, _ = weights["W1"].shape
        c = _Router()
        c.d, c.h, c.ff, c.n_blocks = int(d), int(h), int(ff), int(L)
        for k in ROUTER_KEYS:
            setattr(c, k, _ptr(weights[k]))
        self._c = c

    def forward(self, hidden, R: int, row_idx=None, n_rows_dev=None, logits=None, switch=None, refine_mask=None,
                stream=None, check: bool = True):
        """rstitch_router_forward; returns (logits float32 [R, 2], switch uint8 [R])."""
        import torch
        if logits is None:
            logits = torch.zeros((max(R, 1), 2), dtype=torch.float32, device=hidden.device)
        if switch is None:
            switch = torch.full((max(R, 1),), 255, dtype=torch.uint8, device=hidden.device)
        st = lib().rstitch_router_forward(C.byref(self._c), _ptr(hidden), int(hidden.shape[0]), _ptr(row_idx),
                                          _ptr(n_rows_dev), int(R), _ptr(logits), _ptr(switch), _ptr(refine_mask),
                                          _stream_ptr(stream))
        if not check:
            return st
        if st != 0:
            raise RstitchError(st, "rstitch_router_forward")
        return logits, switch

    def route(self, hidden, R: int, row_idx, route_mask, llm_idx, llm_count, n_rows_dev=None, logits=None,
              switch=None, stream=None, check: bool = True, alg1_tail=None, tok=None, n_seq_dev=None):
        """rstitch_router_route: the router on the rows row_idx names, route_mask refined in place and
        compacted into llm_idx / llm_count by the same launch; returns (logits, switch).  With alg1_tail
        (and tok, the SLM call's tokens) it is rstitch_router_route_alg1: the launch goes on with
        Algorithm 1's decision block for the SLM's batch on the refined mask."""
        import torch
        if logits is None:
            logits = torch.zeros((max(R, 1), 2), dtype=torch.float32, device=hidden.device)
        if switch is None:
            switch = torch.full((max(R, 1),), 255, dtype=torch.uint8, device=hidden.device)
        if alg1_tail is not None:
            st = lib().rstitch_router_route_alg1(C.byref(self._c), _ptr(hidden), int(hidden.shape[0]), _ptr(n_seq_dev),
                                                 _ptr(row_idx), _ptr(n_rows_dev), int(R), _ptr(logits), _ptr(switch),
                                                 _ptr(route_mask), _ptr(llm_idx), _ptr(llm_count), _ptr(tok),
                                                 C.byref(alg1_tail), _stream_ptr(stream))
            if not check:
                return st
            if st != 0:
                raise RstitchError(st, "rstitch_router_route_alg1")
            return logits, switch
        st = lib().rstitch_router_route(C.byref(self._c), _ptr(hidden), int(hidden.shape[0]), _ptr(row_idx),
                                        _ptr(n_rows_dev), int(R), _ptr(logits), _ptr(switch), _ptr(route_mask),
                                        _ptr(llm_idx), _ptr(llm_count), _stream_ptr(stream))
        if not check:
            return st
        if st != 0:
            raise RstitchError(st, "rstitch_router_route")
        return logits, switch
