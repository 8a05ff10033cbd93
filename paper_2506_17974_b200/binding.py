"""ctypes binding of liblqsgd.so (the C ABI declared in include/lqsgd.h).

Argument marshalling only: every step of the LQ-SGD round runs in the library's CUDA kernels.
PyTorch appears here as the owner of device memory (the workspace, gradients, outputs) and of
the CUDA stream.  There is no CPU fallback: if the shared library is missing or a call fails,
an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblqsgd.so")

# lqsgd_state
STATE_E, STATE_Q, STATE_P_RAW, STATE_P, STATE_P_BAR, STATE_Q_W, STATE_CODES_P, STATE_CODES_Q, STATE_SCALES = range(9)
STATUS_DEPENDENT_COLUMN, STATUS_ZERO_SCALE_P, STATUS_ZERO_SCALE_Q, STATUS_NONFINITE = 1, 2, 4, 8
FLAG_HOST_STAGING = 1
FLAG_REGISTER_PATH = 2
FLAG_AVERAGE_VALUES = 4
FLAG_QUANTIZE_VECTORS = 8
FLAG_COLUMN_SCALES = 16
FLAG_ONE_LAUNCH = 32
FLAG_GUARD_WORDS = 64
STATUS_TIMEOUT = 16
N_PHASES = 5
XCHG_SCALES_P, XCHG_SCALES_Q, XCHG_STREAMS_P, XCHG_STREAMS_Q, XCHG_VECTORS = range(5)
PHASE_NAMES = ("pass1", "finish_p", "pass2", "finish_q", "pass3")

ERR_INVALID_ARG, ERR_BAD_SHAPE, ERR_WORKSPACE_TOO_SMALL, ERR_MISALIGNED = -1, -2, -3, -4
ERR_CUDA, ERR_NO_STAGING, ERR_OUT_OF_RANGE = -5, -6, -7
ERR_TOO_LARGE = -8
ERR_CAPTURE = -9
ERR_PLAN = -10
NOALLOC_MAX_ROWS = 65536

EXPORTED = [
    "lqsgd_workspace_bytes", "lqsgd_create", "lqsgd_step", "lqsgd_step_update", "lqsgd_step_host", "lqsgd_payload_bytes",
    "lqsgd_payload", "lqsgd_payload_layout", "lqsgd_get_state", "lqsgd_set_state", "lqsgd_status", "lqsgd_step_stats",
    "lqsgd_orthonormalize_noalloc",
    "lqsgd_round_begin", "lqsgd_round_pack", "lqsgd_round_reduce", "lqsgd_round_end", "lqsgd_exchange_view",
    "lqsgd_launches_per_step", "lqsgd_set_phase_events", "lqsgd_release_graph_tables", "lqsgd_test_expire_wait", "lqsgd_round_timeline", "lqsgd_check_guards", "lqsgd_plan_check", "lqsgd_test_plan_defect", "lqsgd_destroy", "lqsgd_strerror", "lqsgd_last_cuda_error", "lqsgd_version",
]


class Shape(C.Structure):
    _fields_ = [("rows", C.c_int32), ("cols", C.c_int32)]


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("rank", C.c_int32), ("bits_p", C.c_int32),
                ("bits_q", C.c_int32), ("alpha", C.c_float), ("workers", C.c_int32),
                ("seed", C.c_uint64), ("flags", C.c_uint32), ("world_workers", C.c_int32), ("power_iters", C.c_int32)]


class LayerLayout(C.Structure):
    _fields_ = [("is_matrix", C.c_int32), ("rank_eff", C.c_int32), ("scale_offset", C.c_uint64),
                ("p_offset", C.c_uint64), ("p_bytes", C.c_uint64), ("q_offset", C.c_uint64),
                ("q_bytes", C.c_uint64), ("vec_offset", C.c_uint64), ("vec_bytes", C.c_uint64)]


class LayerStats(C.Structure):
    _fields_ = [("status", C.c_uint32), ("rank_eff", C.c_int32), ("scale_p", C.c_float), ("scale_q", C.c_float),
                ("pivot_ratio", C.c_float), ("pad_", C.c_uint32), ("codes_p", C.c_uint64), ("codes_q", C.c_uint64),
                ("near_p", C.c_uint64), ("near_q", C.c_uint64), ("payload_bytes", C.c_uint64)]


class LqsgdError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"lqsgd error {code}: {text}")
        self.code = code


_lib = None


def load_library() -> C.CDLL:
    """Loads liblqsgd.so (built in-tree by __graft_entry__.build()); raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} not found: build the CUDA library first (no CPU fallback exists)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    lib.lqsgd_workspace_bytes.argtypes = [C.POINTER(Shape), i32, C.POINTER(Config), C.POINTER(sz)]
    lib.lqsgd_create.argtypes = [C.POINTER(Shape), i32, C.POINTER(Config), vp, sz, C.POINTER(vp)]
    lib.lqsgd_step.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp]
    lib.lqsgd_step_update.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.c_float, vp]
    lib.lqsgd_step_host.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp, vp]
    lib.lqsgd_round_begin.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.c_float, vp]
    lib.lqsgd_round_pack.argtypes = [vp, i32, vp]
    lib.lqsgd_round_reduce.argtypes = [vp, i32, vp, i32, vp]
    lib.lqsgd_round_end.argtypes = [vp, vp]
    lib.lqsgd_exchange_view.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(sz)]
    lib.lqsgd_payload_bytes.argtypes = [vp, C.POINTER(sz)]
    lib.lqsgd_payload.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(sz)]
    lib.lqsgd_payload_layout.argtypes = [vp, i32, C.POINTER(LayerLayout)]
    lib.lqsgd_get_state.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.lqsgd_set_state.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.lqsgd_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
    lib.lqsgd_step_stats.argtypes = [vp, i32, C.POINTER(LayerStats), vp]
    lib.lqsgd_launches_per_step.argtypes = [vp, C.POINTER(i32)]
    lib.lqsgd_orthonormalize_noalloc.argtypes = [vp, vp, i32, i32, vp, vp]
    lib.lqsgd_set_phase_events.argtypes = [vp, C.POINTER(vp)]
    lib.lqsgd_release_graph_tables.argtypes = [vp]
    lib.lqsgd_test_expire_wait.argtypes = [vp, i32, i32, C.c_uint32]
    lib.lqsgd_round_timeline.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(i32), vp]
    lib.lqsgd_check_guards.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64), vp]
    lib.lqsgd_plan_check.argtypes = [vp, i32, vp, i32, C.c_char_p, C.c_size_t]
    lib.lqsgd_test_plan_defect.argtypes = [i32]
    lib.lqsgd_destroy.argtypes = [vp]
    lib.lqsgd_destroy.restype = None
    lib.lqsgd_strerror.argtypes = [C.c_int]
    lib.lqsgd_strerror.restype = C.c_char_p
    lib.lqsgd_last_cuda_error.restype = C.c_char_p
    lib.lqsgd_version.restype = C.c_int
    _lib = lib
    return lib


def _check(rc: int) -> None:
    if rc != 0:
        lib = load_library()
        text = lib.lqsgd_strerror(rc).decode()
        if rc == ERR_CUDA:
            text += " (" + lib.lqsgd_last_cuda_error().decode() + ")"
        raise LqsgdError(rc, text)


def _shapes(layers: Sequence[Tuple[int, int]]):
    arr = (Shape * len(layers))()
    for i, (n, m) in enumerate(layers):
        arr[i].rows, arr[i].cols = int(n), int(m)
    return arr


def make_config(rank: int, bits_p: int, bits_q: int, alpha: float, workers: int, seed: int = 0,
                flags: int = 0, world_workers: int = 0, power_iters: int = 0) -> Config:
    return Config(C.sizeof(Config), rank, bits_p, bits_q, alpha, workers, seed, flags, world_workers, power_iters)


def orthonormalize_noalloc(p_in: torch.Tensor, p_out: torch.Tensor, status: Optional[torch.Tensor] = None,
                           rows: Optional[int] = None, rank: Optional[int] = None) -> None:
    """Orthonormalises the columns of the fp32 device matrix p_in (rows x rank, contiguous) into
    p_out without any workspace: for callers that cannot allocate device memory.  The library's
    built-in scratch is shared by all calls on a device, so keep calls ordered on one stream.
    `status`, if given, is a one-element int32/uint32 device tensor that receives status bits.
    rows / rank default to p_in's shape (they can be overridden to exercise the size check)."""
    n = p_in.shape[0] if rows is None else rows
    r = p_in.shape[1] if rank is None else rank
    s = torch.cuda.current_stream(p_in.device)
    _check(load_library().lqsgd_orthonormalize_noalloc(
        C.c_void_p(p_in.data_ptr()), C.c_void_p(p_out.data_ptr()), n, r,
        C.c_void_p(status.data_ptr() if status is not None else 0), C.c_void_p(s.cuda_stream)))


def workspace_bytes(layers, cfg: Config) -> int:
    out = C.c_size_t(0)
    _check(load_library().lqsgd_workspace_bytes(_shapes(layers), len(layers), C.byref(cfg), C.byref(out)))
    return out.value


def test_plan_defect(kind: int) -> None:
    """Test support: the next plan_check of this thread damages its private tables first (see the header)."""
    _check(load_library().lqsgd_test_plan_defect(kind))


def plan_check(layers, cfg: Config, sm_count: int = 148) -> str:
    """Host-only self-check of the work tables for this configuration (lqsgd_plan_check): "" when every invariant
    holds, else the description of the first one that fails; raises for an invalid configuration."""
    msg = C.create_string_buffer(512)
    rc = load_library().lqsgd_plan_check(_shapes(layers), len(layers), C.byref(cfg), sm_count, msg, len(msg))
    if rc == ERR_PLAN:
        return msg.value.decode() or "plan check failed"
    _check(rc)
    return ""


class LQSGD:
    """One LQ-SGD compressor (Algorithm 1 state for a list of layers and W workers) on a CUDA device."""

    def __init__(self, layers: Sequence[Tuple[int, int]], rank: int, bits_p: int, bits_q: Optional[int] = None,
                 alpha: float = 127.0, workers: int = 1, seed: int = 0, host_staging: bool = False,
                 device: str = "cuda:0", register_path: bool = False, world_workers: int = 0,
                 average: str = "codes", quantize_vectors: bool = False, power_iters: int = 1,
                 column_scales: bool = False, one_launch: bool = False, guard_words: bool = False):
        self.lib = load_library()
        self.layers = [(int(n), int(m)) for n, m in layers]
        self.rank, self.bits_p = rank, bits_p
        self.bits_q = bits_p if bits_q is None else bits_q
        self.alpha, self.W = float(alpha), workers
        if average not in ("codes", "values"):
            raise ValueError("average must be 'codes' (Algorithm 1) or 'values'")
        self.average = average
        self.quantize_vectors = bool(quantize_vectors) and bits_p != 32
        self.power_iters = max(1, int(power_iters))
        self.column_scales = bool(column_scales)
        self.device = torch.device(device)
        self.cfg = make_config(rank, self.bits_p, self.bits_q, alpha, workers, seed,
                               (FLAG_HOST_STAGING if host_staging else 0)
                               | (FLAG_REGISTER_PATH if register_path else 0)
                               | (FLAG_AVERAGE_VALUES if average == "values" else 0)
                               | (FLAG_QUANTIZE_VECTORS if quantize_vectors else 0)
                               | (FLAG_COLUMN_SCALES if column_scales else 0)
                               | (FLAG_ONE_LAUNCH if one_launch else 0)
                               | (FLAG_GUARD_WORDS if guard_words else 0), world_workers, power_iters)
        nbytes = workspace_bytes(self.layers, self.cfg)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            ctx = C.c_void_p()
            _check(self.lib.lqsgd_create(_shapes(self.layers), len(self.layers), C.byref(self.cfg),
                                         C.c_void_p(self._ws_ptr), nbytes, C.byref(ctx)))
        self.ctx = ctx
        self.workspace_nbytes = nbytes
        out = C.c_size_t(0)
        _check(self.lib.lqsgd_payload_bytes(self.ctx, C.byref(out)))
        self.payload_nbytes = out.value
        n = C.c_int32(0)
        _check(self.lib.lqsgd_launches_per_step(self.ctx, C.byref(n)))
        self.launches_per_step = n.value
        self._keep = None

    # -- lifetime
    def close(self):
        if getattr(self, "ctx", None):
            self.lib.lqsgd_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def r_eff(self, layer: int) -> int:
        n, m = self.layers[layer]
        return min(self.rank, n, m)

    def is_matrix(self, layer: int) -> bool:
        n, m = self.layers[layer]
        return n > 1 and m > 1

    # -- the round
    def make_pointer_arrays(self, grads: Sequence[Sequence[torch.Tensor]], ghat: Sequence[torch.Tensor]):
        """ctypes pointer arrays for step(): grads[w][l] worker-major, ghat[l]."""
        nl = len(self.layers)
        g = (C.c_void_p * (self.W * nl))()
        for w in range(self.W):
            for l in range(nl):
                g[w * nl + l] = grads[w][l].data_ptr()
        h = (C.c_void_p * nl)()
        for l in range(nl):
            h[l] = ghat[l].data_ptr()
        return g, h

    def step_ptrs(self, g_arr, h_arr, stream: Optional[torch.cuda.Stream] = None) -> None:
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        _check(self.lib.lqsgd_step(self.ctx, g_arr, h_arr, C.c_void_p(s.cuda_stream)))

    def round_timeline(self) -> List[int]:
        """Global-timer stamps (ns) of the last round of a one-launch context, [] for a multi-kernel one."""
        buf = (C.c_uint64 * 24)()
        n = C.c_int32(0)
        _check(self.lib.lqsgd_round_timeline(self.ctx, buf, C.byref(n), self._stream_ptr()))
        return [int(buf[i]) for i in range(n.value)]

    def check_guards(self) -> Tuple[int, int]:
        """(guard words changed, byte offset of the first or -1) for a context created with guard_words=True."""
        bad, first = C.c_int64(0), C.c_int64(0)
        _check(self.lib.lqsgd_check_guards(self.ctx, C.byref(bad), C.byref(first), self._stream_ptr()))
        return bad.value, first.value

    def release_graph_tables(self) -> None:
        """Every graph captured from this context's steps is gone: its pointer tables may be reused."""
        _check(self.lib.lqsgd_release_graph_tables(self.ctx))

    def test_expire_wait(self, pass_: int, stage: int, wait_limit: int = 256) -> None:
        """Test support: the next step's pass `pass_` leaves out one stage of copies on CTA 0 and every bounded
        wait gives up after wait_limit polls, so that LQSGD_STATUS_TIMEOUT is raised without any fault."""
        _check(self.lib.lqsgd_test_expire_wait(self.ctx, pass_, stage, wait_limit))

    def set_phase_events(self, events: Optional[Sequence[torch.cuda.Event]]) -> None:
        """Asks the next step to record N_PHASES + 1 caller-owned CUDA events at its phase boundaries."""
        if events is None:
            _check(self.lib.lqsgd_set_phase_events(self.ctx, None))
            return
        assert len(events) == N_PHASES + 1
        for e in events:
            if not e.cuda_event:          # torch creates the handle lazily, on the first record
                e.record(torch.cuda.current_stream(self.device))
        arr =(C.c_void_p * len(events))(*[e.cuda_event for e in events])
        _check(self.lib.lqsgd_set_phase_events(self.ctx, arr))

    def step(self, grads, ghat, stream: Optional[torch.cuda.Stream] = None) -> None:
        """One round of Algorithm 1 on device tensors grads[w][l]; writes ghat[l]."""
        g, h = self.make_pointer_arrays(grads, ghat)
        self.step_ptrs(g, h, stream)

    def step_update(self, grads, ghat, weights, lr: float, stream: Optional[torch.cuda.Stream] = None) -> None:
        """One round plus the model update w <- w - lr * G_hat (Algorithm 1, last line) fused into the
        reconstruction pass.  weights[l] (device tensors, or None entries) are updated in place;
        ghat may be None or hold None entries: G_hat of those layers is not materialised."""
        nl = len(self.layers)
        g = (C.c_void_p * (self.W * nl))()
        for w in range(self.W):
            for l in range(nl):
                g[w * nl + l] = grads[w][l].data_ptr()
        h = None
        if ghat is not None:
            h = (C.c_void_p * nl)(*[(t.data_ptr() if t is not None else None) for t in ghat])
        wt = (C.c_void_p * nl)(*[(t.data_ptr() if t is not None else None) for t in weights])
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        _check(self.lib.lqsgd_step_update(self.ctx, g, h, wt, C.c_float(lr), C.c_void_p(s.cuda_stream)))

    # -- the round in pieces (workers on several GPUs; see paper_2506_17974_b200/distributed.py)
    def round_begin(self, grads, ghat, weights=None, lr: float = 0.0) -> None:
        nl = len(self.layers)
        g = (C.c_void_p * (self.W * nl))()
        for w in range(self.W):
            for l in range(nl):
                g[w * nl + l] = grads[w][l].data_ptr()
        h = (C.c_void_p * nl)(*[(t.data_ptr() if t is not None else None) for t in ghat]) if ghat is not None else None
        wt = (C.c_void_p * nl)(*[(t.data_ptr() if t is not None else None) for t in weights]) if weights is not None else None
        _check(self.lib.lqsgd_round_begin(self.ctx, g, h, wt, C.c_float(lr), self._stream_ptr()))

    def round_pack(self, which: int) -> None:
        _check(self.lib.lqsgd_round_pack(self.ctx, which, self._stream_ptr()))

    def round_reduce(self, which: int, gathered: torch.Tensor, n_ranks: int) -> None:
        _check(self.lib.lqsgd_round_reduce(self.ctx, which, C.c_void_p(gathered.data_ptr()), n_ranks, self._stream_ptr()))

    def round_end(self) -> None:
        _check(self.lib.lqsgd_round_end(self.ctx, self._stream_ptr()))

    def exchange_view(self, which: int) -> torch.Tensor:
        """The exchange buffer `which` (XCHG_*) as a tensor aliasing the workspace: fp32 scales or uint8 streams."""
        ptr, nb = C.c_void_p(), C.c_size_t(0)
        _check(self.lib.lqsgd_exchange_view(self.ctx, which, C.byref(ptr), C.byref(nb)))
        off = ptr.value - self.workspace.data_ptr()
        raw = self.workspace[off:off + nb.value]
        return raw.view(torch.float32) if which in (XCHG_SCALES_P, XCHG_SCALES_Q, XCHG_VECTORS) else raw

    def step_host(self, grads, ghat, payload: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None) -> None:
        """Same round on HOST tensors (copies in, runs, copies G_hat and payloads out, synchronises)."""
        g, h = self.make_pointer_arrays(grads, ghat)
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        pp = C.c_void_p(payload.data_ptr()) if payload is not None else C.c_void_p(0)
        _check(self.lib.lqsgd_step_host(self.ctx, g, h, pp, C.c_void_p(s.cuda_stream)))

    # -- results and state
    def _stream_ptr(self):
        return C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)

    def payload(self, worker: int) -> torch.Tensor:
        """Copy of worker's payload bytes (uint8 device tensor)."""
        ptr, nb = C.c_void_p(), C.c_size_t(0)
        _check(self.lib.lqsgd_payload(self.ctx, worker, C.byref(ptr), C.byref(nb)))
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + nb.value].clone()

    def payload_layout(self, layer: int) -> LayerLayout:
        out = LayerLayout()
        _check(self.lib.lqsgd_payload_layout(self.ctx, layer, C.byref(out)))
        return out

    def _state_shape(self, which: int, layer: int):
        if not 0 <= layer < len(self.layers) or which not in range(9):
            return (1,), torch.float32          # the library reports the bad index
        n, m = self.layers[layer]
        r = self.r_eff(layer)
        return {STATE_E: ((n, m), torch.float32), STATE_Q: ((m, r), torch.float32),
                STATE_P_RAW: ((n, r), torch.float32), STATE_P: ((n, r), torch.float32),
                STATE_P_BAR: ((n, r), torch.float32), STATE_Q_W: ((m, r), torch.float32),
                STATE_CODES_P: ((n, r), torch.uint8), STATE_CODES_Q: ((m, r), torch.uint8),
                STATE_SCALES: (((2, r) if self.column_scales else (2,)), torch.float32)}[which]

    def get_state(self, which: int, layer: int, worker: int = 0) -> torch.Tensor:
        shape, dt = self._state_shape(which, layer)
        out = torch.empty(shape, dtype=dt, device=self.device)
        _check(self.lib.lqsgd_get_state(self.ctx, which, layer, worker, C.c_void_p(out.data_ptr()), self._stream_ptr()))
        return out

    def set_state(self, which: int, layer: int, worker: int, value: torch.Tensor) -> None:
        shape, dt = self._state_shape(which, layer)
        v = value.to(device=self.device, dtype=dt).contiguous()
        assert tuple(v.shape) == tuple(shape), (v.shape, shape)
        _check(self.lib.lqsgd_set_state(self.ctx, which, layer, worker, C.c_void_p(v.data_ptr()), self._stream_ptr()))
        torch.cuda.current_stream(self.device).synchronize()      # v may be a temporary

    def step_stats(self, layer: int) -> dict:
        """Figures of the last round for one layer (lqsgd_layer_stats as a dict)."""
        st = LayerStats()
        _check(self.lib.lqsgd_step_stats(self.ctx, layer, C.byref(st), self._stream_ptr()))
        return {name: getattr(st, name) for name, _ in LayerStats._fields_ if name != "pad_"}

    def status(self) -> List[int]:
        flags = (C.c_uint32 * len(self.layers))()
        _check(self.lib.lqsgd_status(self.ctx, flags, self._stream_ptr()))
        return list(flags)
