"""ctypes binding of ``libdeltalog.so``: argument marshalling only.

Every step of the decode / append / merge / eager path runs in the CUDA kernels behind the C ABI
declared in ``include/deltalog.h``; this module turns torch tensors into raw pointers, passes the
current CUDA stream and raises on a non-zero return code.  There is no CPU fallback: if the shared
library is missing or cannot be loaded, importing the symbols raises.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from pathlib import Path
from typing import Optional

import torch

GDN, KDA, RWKV6, LINATTN, RETNET, GLA = 0, 1, 2, 3, 4, 5
HINT_BASE_UNTOUCHED, HINT_SLOTS_STABLE, HINT_WALK_DOWN = 1, 2, 4
_DELTA_RULE = (GDN, KDA)            # b = beta (v - S'^T k): U log in fp32
_VEC_DECAY = (KDA, RWKV6, GLA)      # one log-decay per key channel
F32, BF16 = 0, 1
STATUS_LOG_FULL, STATUS_BAD_SLOT, STATUS_TIMEOUT = 1, 2, 4
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_CAP_RANGE, ERR_CUDA, ERR_STATIC_LIMIT = 0, 1, 2, 3, 4, 5
STATIC_STAGING_BYTES = 8 << 20

_TORCH_TO_DT = {torch.float32: F32, torch.bfloat16: BF16}
_DT_TO_TORCH = {F32: torch.float32, BF16: torch.bfloat16}

LIB_PATH = Path(__file__).resolve().parent / "libdeltalog.so"

EXPORTS = (
    "deltalog_decode_step", "deltalog_decode_steps", "deltalog_decode_merge_step", "deltalog_merge", "deltalog_reset_slots", "deltalog_eager_step", "deltalog_decode_step_host",
    "deltalog_decode_step_host_static", "deltalog_decode_step_host_overlapped",
    "deltalog_status_string", "deltalog_version", "deltalog_build_id", "deltalog_launch_count",
)


class DeltalogError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (code {code})")


class _Desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("op", "num_slots", "H", "d_k", "d_v", "cap", "io_dtype", "klog_dtype", "ulog_dtype")] + \
               [("scale", ctypes.c_float), ("H_qk", ctypes.c_int32), ("hints", ctypes.c_int32), ("base_dtype", ctypes.c_int32)]


class _State(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("S_base", "K_log", "U_log", "decay_log", "log_len", "status")]


class _Staging(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("q", "k", "v", "g", "beta", "out")] + [("packed", ctypes.c_int32)]


class _Lane(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("copy_in_stream", "compute_stream", "copy_out_stream", "in_done", "compute_done", "out_done")]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load ``libdeltalog.so`` (built by ``paper_2608_15533_b200.build``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2608_15533_b200.build` "
                "(there is no fallback path)")
        lib = ctypes.CDLL(str(LIB_PATH))
        vp, i32 = ctypes.c_void_p, ctypes.c_int32
        lib.deltalog_decode_step.restype = ctypes.c_int
        lib.deltalog_decode_step.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(_State)] + [vp] * 7 + [i32, vp, vp]
        lib.deltalog_decode_steps.restype = ctypes.c_int
        lib.deltalog_decode_steps.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(_State)] + [vp] * 7 + [i32, i32, vp, vp]
        lib.deltalog_decode_merge_step.restype = ctypes.c_int
        lib.deltalog_decode_merge_step.argtypes = lib.deltalog_decode_step.argtypes
        lib.deltalog_merge.restype = ctypes.c_int
        lib.deltalog_merge.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(_State), vp, i32, i32, vp]
        lib.deltalog_reset_slots.restype = ctypes.c_int
        lib.deltalog_reset_slots.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(_State), vp, i32, vp, vp]
        lib.deltalog_eager_step.restype = ctypes.c_int
        lib.deltalog_eager_step.argtypes = [ctypes.POINTER(_Desc)] + [vp] * 8 + [i32, vp, vp, vp]
        lib.deltalog_decode_step_host.restype = ctypes.c_int
        lib.deltalog_decode_step_host.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(_State),
                                                  ctypes.POINTER(_Staging)] + [vp] * 7 + [i32, vp, vp]
        lib.deltalog_decode_step_host_static.restype = ctypes.c_int
        lib.deltalog_decode_step_host_static.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(_State)] + [vp] * 7 + [i32, vp, vp]
        lib.deltalog_decode_step_host_overlapped.restype = ctypes.c_int
        lib.deltalog_decode_step_host_overlapped.argtypes = [ctypes.POINTER(_Desc), ctypes.POINTER(_State),
                                                             ctypes.POINTER(_Staging), ctypes.POINTER(_Lane)] + [vp] * 7 + [i32, vp]
        lib.deltalog_status_string.restype = ctypes.c_char_p
        lib.deltalog_status_string.argtypes = [ctypes.c_int]
        lib.deltalog_version.restype = ctypes.c_int
        lib.deltalog_build_id.restype = ctypes.c_char_p
        lib.deltalog_launch_count.restype = ctypes.c_uint64
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load_library().deltalog_status_string(int(code)).decode()


def version() -> int:
    return int(load_library().deltalog_version())


def build_id() -> str:
    """Identifier of the sources the loaded library was built from (see ``build.source_id``)."""
    return load_library().deltalog_build_id().decode()


def launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(load_library().deltalog_launch_count())


@dataclass
class Desc:
    """Mirror of ``deltalog_desc``."""

    op: int
    num_slots: int
    H: int
    d_k: int
    d_v: int
    cap: int
    io_dtype: int = BF16
    klog_dtype: Optional[int] = None   # default: io_dtype
    ulog_dtype: Optional[int] = None   # default: F32 for GDN / KDA, io_dtype where b = v
    scale: float = 1.0
    H_qk: int = 0                      # query/key heads (0 = H); a divisor of H groups value heads
    hints: int = 0                     # HINT_* bits (promises by the caller, see the header)
    base_dtype: int = F32              # dtype of the dense state; BF16 = the 16-bit state (needs io_dtype BF16)

    def __post_init__(self):
        if self.klog_dtype is None:
            self.klog_dtype = self.io_dtype
        if self.ulog_dtype is None:
            self.ulog_dtype = F32 if self.op in _DELTA_RULE else self.io_dtype

    @property
    def d_lambda(self) -> int:
        return self.d_k if self.op in _VEC_DECAY else 1

    def c_struct(self) -> _Desc:
        key = (self.op, self.num_slots, self.H, self.d_k, self.d_v, self.cap, self.io_dtype,
               self.klog_dtype, self.ulog_dtype, float(self.scale), int(self.H_qk), int(self.hints),
               int(self.base_dtype))
        cached = self.__dict__.get("_c")
        if cached is None or cached[0] != key:
            cached = (key, _Desc(*key))
            self.__dict__["_c"] = cached
        return cached[1]


class State:
    """Device tensors of the physical state (base, log, snapshots, lengths, status word)."""

    def __init__(self, desc: Desc, S_base: torch.Tensor, device=None):
        device = S_base.device if device is None else device
        n, H, cap = desc.num_slots, desc.H, desc.cap
        assert S_base.shape == (n, H, desc.d_k, desc.d_v) and S_base.dtype == _DT_TO_TORCH[desc.base_dtype]
        self.desc = desc
        self.S_base = S_base.contiguous()
        self.K_log = torch.zeros(n, H, cap, desc.d_k, dtype=_DT_TO_TORCH[desc.klog_dtype], device=device)
        self.U_log = torch.zeros(n, H, cap, desc.d_v, dtype=_DT_TO_TORCH[desc.ulog_dtype], device=device)
        self.decay_log = torch.zeros(n, H, cap, desc.d_lambda, dtype=torch.float32, device=device)
        self.log_len = torch.zeros(n, H, dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def c_struct(self) -> _State:
        ptrs = (self.S_base.data_ptr(), self.K_log.data_ptr(), self.U_log.data_ptr(),
                self.decay_log.data_ptr(), self.log_len.data_ptr(), self.status.data_ptr())
        cached = getattr(self, "_c", None)
        if cached is None or cached[0] != ptrs:
            cached = (ptrs, _State(*ptrs))
            self._c = cached
        return cached[1]

    def log_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in (self.K_log, self.U_log, self.decay_log))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the C ABI must be contiguous"
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise DeltalogError(rc, where)


def decode_step(desc: Desc, state: State, q, k, v, g, beta=None, u_bonus=None, slot_idx=None, out=None,
                stream=None) -> torch.Tensor:
    """``deltalog_decode_step``: one token for ``B = q.shape[0]`` rows; returns ``out [B,H,d_v]``."""
    B = q.shape[0]
    if out is None:
        out = torch.empty(B, desc.H, desc.d_v, dtype=q.dtype, device=q.device)
    d, s = desc.c_struct(), state.c_struct()
    rc = load_library().deltalog_decode_step(
        ctypes.byref(d), ctypes.byref(s), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(u_bonus),
        _ptr(slot_idx), B, _ptr(out), _stream(stream))
    _check(rc, "deltalog_decode_step")
    return out


def decode_steps(desc: Desc, state: State, q, k, v, g, beta=None, u_bonus=None, slot_idx=None, out=None,
                 stream=None) -> torch.Tensor:
    """``deltalog_decode_steps``: ``T = q.shape[1]`` consecutive tokens per row (token tensors
    ``[B,T,H,d]``) with one read of the base tile; returns ``out [B,T,H,d_v]``."""
    B, T = q.shape[0], q.shape[1]
    if out is None:
        out = torch.empty(B, T, desc.H, desc.d_v, dtype=q.dtype, device=q.device)
    d, s = desc.c_struct(), state.c_struct()
    rc = load_library().deltalog_decode_steps(
        ctypes.byref(d), ctypes.byref(s), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(u_bonus),
        _ptr(slot_idx), B, T, _ptr(out), _stream(stream))
    _check(rc, "deltalog_decode_steps")
    return out


def decode_merge_step(desc: Desc, state: State, q, k, v, g, beta=None, u_bonus=None, slot_idx=None, out=None,
                      stream=None) -> torch.Tensor:
    """``deltalog_decode_merge_step``: one token for every row AND materialisation of its state (the
    merge step of the paper's cycle); returns ``out [B,H,d_v]``."""
    B = q.shape[0]
    if out is None:
        out = torch.empty(B, desc.H, desc.d_v, dtype=q.dtype, device=q.device)
    d, s = desc.c_struct(), state.c_struct()
    rc = load_library().deltalog_decode_merge_step(
        ctypes.byref(d), ctypes.byref(s), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(u_bonus),
        _ptr(slot_idx), B, _ptr(out), _stream(stream))
    _check(rc, "deltalog_decode_merge_step")
    return out


def merge(desc: Desc, state: State, slot_idx=None, n: Optional[int] = None, only_if_full: bool = False,
          stream=None) -> None:
    """``deltalog_merge`` over the listed slots (all ``num_slots`` when ``slot_idx`` is None)."""
    if n is None:
        n = desc.num_slots if slot_idx is None else slot_idx.numel()
    d, s = desc.c_struct(), state.c_struct()
    rc = load_library().deltalog_merge(ctypes.byref(d), ctypes.byref(s), _ptr(slot_idx), int(n),
                                       int(bool(only_if_full)), _stream(stream))
    _check(rc, "deltalog_merge")


def reset_slots(desc: Desc, state: State, slot_idx=None, n: Optional[int] = None, S_init=None, stream=None) -> None:
    """``deltalog_reset_slots``: empty the logs of the listed slots (all when ``slot_idx`` is None) and,
    with ``S_init [n,H,d_k,d_v]`` fp32, install new base states (prefill hand-off)."""
    assert S_init is None or S_init.dtype == torch.float32
    if n is None:
        n = desc.num_slots if slot_idx is None else slot_idx.numel()
    d, s = desc.c_struct(), state.c_struct()
    rc = load_library().deltalog_reset_slots(ctypes.byref(d), ctypes.byref(s), _ptr(slot_idx), int(n),
                                             _ptr(S_init), _stream(stream))
    _check(rc, "deltalog_reset_slots")


def eager_step(desc: Desc, S: torch.Tensor, q, k, v, g, beta=None, u_bonus=None, slot_idx=None, out=None,
               status=None, stream=None) -> torch.Tensor:
    """``deltalog_eager_step``: the dense comparator; ``S`` (dtype ``desc.base_dtype``) is rewritten in place."""
    assert S.dtype == _DT_TO_TORCH[desc.base_dtype]
    B = q.shape[0]
    if out is None:
        out = torch.empty(B, desc.H, desc.d_v, dtype=q.dtype, device=q.device)
    d = desc.c_struct()
    rc = load_library().deltalog_eager_step(
        ctypes.byref(d), _ptr(S), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(u_bonus),
        _ptr(slot_idx), B, _ptr(out), _ptr(status), _stream(stream))
    _check(rc, "deltalog_eager_step")
    return out


def _packed_views(desc: "Desc", B: int, block: torch.Tensor):
    """q, k, v, g, beta as views into one byte block, each starting on the next 256-byte boundary
    after the previous one ends (the layout the library recognises and copies in one piece)."""
    io = _DT_TO_TORCH[desc.io_dtype]
    esz = torch.empty((), dtype=io).element_size()
    Hqk = desc.H_qk or desc.H
    gshape = (B, desc.H, desc.d_k) if desc.op in _VEC_DECAY else (B, desc.H)
    specs = [("q", (B, Hqk, desc.d_k), io), ("k", (B, Hqk, desc.d_k), io), ("v", (B, desc.H, desc.d_v), io),
             ("g", gshape, torch.float32), ("beta", (B, desc.H), torch.float32)]
    out, off = {}, 0
    for name, shape, dt in specs:
        n = 1
        for x in shape:
            n *= x
        nbytes = n * (esz if dt == io else 4)
        if block is not None:
            out[name] = block[off:off + nbytes].view(dt).view(*shape)
        off = (off + nbytes + 255) // 256 * 256
    return out, off


def packed_host_tokens(desc: "Desc", B: int) -> dict:
    """Pinned host tensors q, k, v, g, beta laid out back to back (256-byte aligned) in one block:
    together with ``HostStaging`` the host-buffer entry points then issue a single copy."""
    _, total = _packed_views(desc, B, None)
    block = torch.empty(total, dtype=torch.uint8).pin_memory()
    views, _ = _packed_views(desc, B, block)
    views["_block"] = block
    return views


class HostStaging:
    """Device staging buffers for ``decode_step_host`` (allocated once, reused every step), carved
    out of one block in the packed layout."""

    def __init__(self, desc: Desc, B: int, device):
        io = _DT_TO_TORCH[desc.io_dtype]
        _, total = _packed_views(desc, B, None)
        self._block = torch.empty(total, dtype=torch.uint8, device=device)
        v, _ = _packed_views(desc, B, self._block)
        self.q, self.k, self.v, self.g, self.beta = v["q"], v["k"], v["v"], v["g"], v["beta"]
        self.out = torch.empty(B, desc.H, desc.d_v, dtype=io, device=device)
        self.packed = False   # set by the caller who also passes ``packed_host_tokens`` buffers

    def c_struct(self) -> _Staging:
        return _Staging(*(t.data_ptr() for t in (self.q, self.k, self.v, self.g, self.beta, self.out)),
                        1 if self.packed else 0)

    def h2d_bytes(self, desc: Desc) -> int:
        ts = [self.q, self.k, self.v, self.g] + ([self.beta] if desc.op in _DELTA_RULE else [])
        return sum(t.numel() * t.element_size() for t in ts)

    def d2h_bytes(self) -> int:
        return self.out.numel() * self.out.element_size()


def decode_step_host(desc: Desc, state: State, staging: HostStaging, host_q, host_k, host_v, host_g,
                     host_beta, host_out, u_bonus=None, slot_idx=None, stream=None) -> None:
    """``deltalog_decode_step_host``: token tensors and ``host_out`` are (pinned) host tensors."""
    for t in (host_q, host_k, host_v, host_g, host_out):
        assert t.device.type == "cpu"
    B = host_q.shape[0]
    d, s, st = desc.c_struct(), state.c_struct(), staging.c_struct()
    rc = load_library().deltalog_decode_step_host(
        ctypes.byref(d), ctypes.byref(s), ctypes.byref(st), _ptr(host_q), _ptr(host_k), _ptr(host_v),
        _ptr(host_g), _ptr(host_beta), _ptr(u_bonus), _ptr(slot_idx), B, _ptr(host_out), _stream(stream))
    _check(rc, "deltalog_decode_step_host")


def decode_step_host_static(desc: Desc, state: State, host_q, host_k, host_v, host_g, host_beta, host_out,
                            u_bonus=None, slot_idx=None, stream=None) -> None:
    """``deltalog_decode_step_host_static``: like ``decode_step_host`` but the device staging area is
    the library's built-in array, for callers that must not allocate device memory.  Raises
    ``DeltalogError`` (code ``ERR_STATIC_LIMIT``) when the token tensors exceed ``STATIC_STAGING_BYTES``.
    Calls on one device share the array: do not let two of them overlap on the GPU."""
    for t in (host_q, host_k, host_v, host_g, host_out):
        assert t.device.type == "cpu"
    B = host_q.shape[0]
    d, s = desc.c_struct(), state.c_struct()
    rc = load_library().deltalog_decode_step_host_static(
        ctypes.byref(d), ctypes.byref(s), _ptr(host_q), _ptr(host_k), _ptr(host_v), _ptr(host_g),
        _ptr(host_beta), _ptr(u_bonus), _ptr(slot_idx), B, _ptr(host_out), _stream(stream))
    _check(rc, "deltalog_decode_step_host_static")


class HostLane:
    """Streams (shared) and one event triple (per staging set) for ``decode_step_host_overlapped``."""

    def __init__(self, copy_in: "torch.cuda.Stream", compute: "torch.cuda.Stream", copy_out: "torch.cuda.Stream"):
        self.copy_in, self.compute, self.copy_out = copy_in, compute, copy_out
        self.in_done, self.compute_done, self.out_done = (torch.cuda.Event() for _ in range(3))
        for ev, st in ((self.in_done, copy_in), (self.compute_done, compute), (self.out_done, copy_out)):
            ev.record(st)  # creates the underlying CUDA event

    def c_struct(self) -> _Lane:
        return _Lane(self.copy_in.cuda_stream, self.compute.cuda_stream, self.copy_out.cuda_stream,
                     self.in_done.cuda_event, self.compute_done.cuda_event, self.out_done.cuda_event)


def decode_step_host_overlapped(desc: Desc, state: State, staging: HostStaging, lane: HostLane, host_q, host_k,
                                host_v, host_g, host_beta, host_out, u_bonus=None, slot_idx=None) -> None:
    """``deltalog_decode_step_host_overlapped``: copy-in, kernel and copy-out on the lane's three streams."""
    B = host_q.shape[0]
    d, s, st, ln = desc.c_struct(), state.c_struct(), staging.c_struct(), lane.c_struct()
    rc = load_library().deltalog_decode_step_host_overlapped(
        ctypes.byref(d), ctypes.byref(s), ctypes.byref(st), ctypes.byref(ln), _ptr(host_q), _ptr(host_k),
        _ptr(host_v), _ptr(host_g), _ptr(host_beta), _ptr(u_bonus), _ptr(slot_idx), B, _ptr(host_out))
    _check(rc, "deltalog_decode_step_host_overlapped")
