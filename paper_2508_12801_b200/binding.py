"""Thin ctypes binding of libmaxscore.so: argument marshalling only.

Every function has the name and argument order of its C entry point (include/maxscore.h) with
the leading ``maxscore_`` dropped.  Tensors are torch CUDA tensors used purely as device memory;
their data pointers go straight into the C ABI.  There is no CPU fallback: if the library cannot
be loaded the import of this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

C_int32 = C.c_int32

F32, BF16 = 0, 1
STAT_NOT_CONVERGED, STAT_NON_FINITE, STAT_INTERNAL = 1, 2, 4
STATUS_NAMES = {0: "OK", 1: "ERR_INVALID_ARG", 2: "ERR_INFEASIBLE", 3: "ERR_WORKSPACE", 4: "ERR_CUDA",
                5: "ERR_NOT_CONVERGED", 6: "ERR_UNSUPPORTED"}


class Params(C.Structure):
    _fields_ = [("T", C.c_int32), ("d_model", C.c_int32), ("E", C.c_int32), ("k", C.c_int32),
                ("capacity_factor", C.c_float), ("capacity", C.c_int32), ("t", C.c_float),
                ("score_mode", C.c_int32), ("quant_shift", C.c_int32), ("tiebreak_seed", C.c_uint32),
                ("max_sweeps", C.c_int32), ("io_dtype", C.c_int32), ("w_gate_layout", C.c_int32),
                ("softtopk_mode", C.c_int32), ("rankscale_beta", C.c_float), ("rankscale_delta", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("status", C.c_uint32), ("capacity", C.c_int32), ("sweeps", C.c_int32),
                ("augmentations", C.c_int32), ("rounds", C.c_int32), ("candidates", C.c_int32),
                ("rerouted", C.c_int32), ("reserved", C.c_int32), ("total_score", C.c_double)]


class DeviceBuffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("hidden", "w_gate", "expert_bias", "logits", "scores", "expert_idx",
                                           "slot_idx", "gate_w", "slot_token", "expert_load", "stats", "xdisp")]


LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmaxscore.so")
EXPORTS = ["maxscore_capacity", "maxscore_workspace_bytes", "maxscore_create", "maxscore_destroy",
           "maxscore_last_cuda_error", "maxscore_route_fwd", "maxscore_dispatch", "maxscore_combine",
           "maxscore_route_bwd", "maxscore_gate", "maxscore_softtopk_fwd", "maxscore_softtopk_bwd",
           "maxscore_assign", "maxscore_index_build", "maxscore_combine_bwd", "maxscore_gate_bwd",
           "maxscore_route_dispatch_host", "maxscore_index_build_noalloc", "maxscore_aux_loss",
           "maxscore_softtopk_bwd_aux", "maxscore_check_internal", "maxscore_launch_count",
           "maxscore_test_raise_internal", "maxscore_assign_iterative", "maxscore_assign_top2_sinkhorn"]


def _load():
    if not os.path.exists(LIB_PATH):
        _build.build()
    lib = C.CDLL(LIB_PATH)
    for name in EXPORTS:
        getattr(lib, name)            # AttributeError here = a declared symbol is missing
    lib.maxscore_capacity.restype = C.c_int32
    lib.maxscore_last_cuda_error.restype = C.c_char_p
    lib.maxscore_destroy.restype = None
    lib.maxscore_launch_count.restype = C.c_longlong
    for name in EXPORTS:
        if name not in ("maxscore_capacity", "maxscore_last_cuda_error", "maxscore_destroy", "maxscore_launch_count"):
            getattr(lib, name).restype = C.c_int
    return lib


_lib = _load()


class MaxScoreError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = _lib.maxscore_last_cuda_error().decode() if status == 4 else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} {detail}".strip())


def _check(status: int, where: str):
    if status != 0:
        raise MaxScoreError(status, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensors must be contiguous"
        return C.c_void_p(t.data_ptr())
    return t


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def make_params(T, d_model, E, k, capacity_factor=1.0, capacity=0, t=1.0, score_mode=0, quant_shift=11,
                tiebreak_seed=0, max_sweeps=0, io_dtype=BF16, w_gate_layout=0, softtopk_mode=0, rankscale_beta=0.0,
                rankscale_delta=0) -> Params:
    return Params(T, d_model, E, k, capacity_factor, capacity, t, score_mode, quant_shift, tiebreak_seed,
                  max_sweeps, io_dtype, w_gate_layout, softtopk_mode, rankscale_beta, rankscale_delta)


def capacity(params: Params) -> int:
    return int(_lib.maxscore_capacity(C.byref(params)))


def workspace_bytes(params: Params) -> int:
    n = C.c_size_t(0)
    _check(_lib.maxscore_workspace_bytes(C.byref(params), C.byref(n)), "maxscore_workspace_bytes")
    return int(n.value)


class Context:
    """Owns the ctx handle and the torch tensor that backs its workspace."""

    def __init__(self, params: Params, device="cuda:0"):
        self.params = params
        nbytes = workspace_bytes(params)
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            self.handle = C.c_void_p()
            _check(_lib.maxscore_create(C.byref(self.handle), C.byref(params), C.c_void_p(base), C.c_size_t(nbytes)),
                   "maxscore_create")
        self.capacity = capacity(params)

    def close(self):
        if self.handle:
            _lib.maxscore_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def create(params: Params, device="cuda:0") -> Context:
    return Context(params, device)


def destroy(ctx: Context):
    ctx.close()


def route_fwd(ctx, hidden, w_gate, expert_bias, logits, scores, expert_idx, slot_idx, gate_w, slot_token,
              expert_load, stats, stream=None):
    _check(_lib.maxscore_route_fwd(ctx.handle, _ptr(hidden), _ptr(w_gate), _ptr(expert_bias), _ptr(logits),
                                   _ptr(scores), _ptr(expert_idx), _ptr(slot_idx), _ptr(gate_w), _ptr(slot_token),
                                   _ptr(expert_load), _ptr(stats), _stream(stream)), "maxscore_route_fwd")


def dispatch(ctx, src, expert_idx, slot_idx, slot_token, dst, stream=None):
    _check(_lib.maxscore_dispatch(ctx.handle, _ptr(src), _ptr(expert_idx), _ptr(slot_idx), _ptr(slot_token),
                                  _ptr(dst), _stream(stream)), "maxscore_dispatch")


def combine(ctx, src, expert_idx, slot_idx, gate_w, dst, accumulate=0, stream=None):
    _check(_lib.maxscore_combine(ctx.handle, _ptr(src), _ptr(expert_idx), _ptr(slot_idx), _ptr(gate_w), _ptr(dst),
                                 C.c_int(accumulate), _stream(stream)), "maxscore_combine")


def route_bwd(ctx, dY, yexp, hidden, w_gate, logits, expert_idx, slot_idx, gate_w, slot_token, dyexp, dgate_w,
              dlogits, dw_gate, dH, stream=None):
    _check(_lib.maxscore_route_bwd(ctx.handle, _ptr(dY), _ptr(yexp), _ptr(hidden), _ptr(w_gate), _ptr(logits),
                                   _ptr(expert_idx), _ptr(slot_idx), _ptr(gate_w), _ptr(slot_token), _ptr(dyexp),
                                   _ptr(dgate_w), _ptr(dlogits), _ptr(dw_gate), _ptr(dH), _stream(stream)),
           "maxscore_route_bwd")


def gate(ctx, hidden, w_gate, expert_bias, logits, stream=None):
    _check(_lib.maxscore_gate(ctx.handle, _ptr(hidden), _ptr(w_gate), _ptr(expert_bias), _ptr(logits),
                              _stream(stream)), "maxscore_gate")


def softtopk_fwd(ctx, logits, scores, stream=None):
    _check(_lib.maxscore_softtopk_fwd(ctx.handle, _ptr(logits), _ptr(scores), _stream(stream)),
           "maxscore_softtopk_fwd")


def softtopk_bwd(ctx, logits, expert_idx, dgate_w, dlogits, stream=None):
    _check(_lib.maxscore_softtopk_bwd(ctx.handle, _ptr(logits), _ptr(expert_idx), _ptr(dgate_w), _ptr(dlogits),
                                      _stream(stream)), "maxscore_softtopk_bwd")


def softtopk_bwd_aux(ctx, logits, expert_idx, dgate_w, dscores_col, dlogits, stream=None):
    _check(_lib.maxscore_softtopk_bwd_aux(ctx.handle, _ptr(logits), _ptr(expert_idx), _ptr(dgate_w), _ptr(dscores_col),
                                          _ptr(dlogits), _stream(stream)), "maxscore_softtopk_bwd_aux")


def aux_loss(ctx, scores, expert_load, lam, loss, dscores_col, stream=None):
    """Eq. 9 and its gradient: loss is a 1-element float64 device tensor, dscores_col an [E] float32 one."""
    _check(_lib.maxscore_aux_loss(ctx.handle, _ptr(scores), _ptr(expert_load), C.c_float(lam), _ptr(loss),
                                  _ptr(dscores_col), _stream(stream)), "maxscore_aux_loss")


def assign(ctx, matrix, expert_idx, expert_load, stats, stream=None):
    _check(_lib.maxscore_assign(ctx.handle, _ptr(matrix), _ptr(expert_idx), _ptr(expert_load), _ptr(stats),
                                _stream(stream)), "maxscore_assign")


def assign_top2_sinkhorn(ctx, scores, sinkhorn_eps, sinkhorn_iters, expert_idx, expert_load, plan, counts, stream=None):
    """Algorithm 1 (k = 2): top-1, then capped Sinkhorn on the residual problem; plan may be None."""
    _check(_lib.maxscore_assign_top2_sinkhorn(ctx.handle, _ptr(scores), C.c_float(sinkhorn_eps), C.c_int32(sinkhorn_iters),
                                              _ptr(expert_idx), _ptr(expert_load), _ptr(plan), _ptr(counts),
                                              _stream(stream)), "maxscore_assign_top2_sinkhorn")


def assign_iterative(ctx, scores, expert_idx, expert_load, counts, stream=None):
    """Top-k with capacity, then greedy rerouting of the dropped pairs; counts is an int32[2] device tensor."""
    _check(_lib.maxscore_assign_iterative(ctx.handle, _ptr(scores), _ptr(expert_idx), _ptr(expert_load), _ptr(counts),
                                          _stream(stream)), "maxscore_assign_iterative")


def index_build(ctx, expert_idx, slot_idx, slot_token, expert_load, stream=None):
    _check(_lib.maxscore_index_build(ctx.handle, _ptr(expert_idx), _ptr(slot_idx), _ptr(slot_token),
                                     _ptr(expert_load), _stream(stream)), "maxscore_index_build")


def combine_bwd(ctx, dY, yexp, expert_idx, slot_idx, gate_w, slot_token, dyexp, dgate_w, stream=None):
    _check(_lib.maxscore_combine_bwd(ctx.handle, _ptr(dY), _ptr(yexp), _ptr(expert_idx), _ptr(slot_idx),
                                     _ptr(gate_w), _ptr(slot_token), _ptr(dyexp), _ptr(dgate_w), _stream(stream)),
           "maxscore_combine_bwd")


def gate_bwd(ctx, hidden, w_gate, dlogits, dw_gate, dH, stream=None):
    _check(_lib.maxscore_gate_bwd(ctx.handle, _ptr(hidden), _ptr(w_gate), _ptr(dlogits), _ptr(dw_gate), _ptr(dH),
                                  _stream(stream)), "maxscore_gate_bwd")


def check_internal(ctx, stream=None) -> int:
    """Reads and clears the context's internal-error flag (synchronises the stream); non-zero = a bounded wait gave up."""
    flag = C.c_uint32(0)
    _check(_lib.maxscore_check_internal(ctx.handle, C.byref(flag), _stream(stream)), "maxscore_check_internal")
    return int(flag.value)


def launch_count(ctx) -> int:
    return int(_lib.maxscore_launch_count(ctx.handle))


def test_raise_internal(ctx, stream=None):
    _check(_lib.maxscore_test_raise_internal(ctx.handle, _stream(stream)), "maxscore_test_raise_internal")


def route_dispatch_host(ctx, hidden_host, w_gate_host, expert_bias_host, dev: DeviceBuffers, expert_idx_host,
                        slot_idx_host, gate_w_host, stats_host, stream=None):
    _check(_lib.maxscore_route_dispatch_host(ctx.handle, _ptr(hidden_host), _ptr(w_gate_host),
                                             _ptr(expert_bias_host), C.byref(dev), _ptr(expert_idx_host),
                                             _ptr(slot_idx_host), _ptr(gate_w_host), _ptr(stats_host),
                                             _stream(stream)), "maxscore_route_dispatch_host")


def index_build_noalloc(T, E, k, C, expert_idx, slot_idx, slot_token, expert_load, stream=None):
    """Index build with no context and no workspace (scratch inside the library); see the header."""
    _check(_lib.maxscore_index_build_noalloc(C_int32(T), C_int32(E), C_int32(k), C_int32(C), _ptr(expert_idx),
                                             _ptr(slot_idx), _ptr(slot_token), _ptr(expert_load), _stream(stream)),
           "maxscore_index_build_noalloc")


# ---- conveniences for callers that keep everything in torch tensors -----------------------------------
def read_stats(stats_tensor: torch.Tensor) -> Stats:
    """Copy a device maxscore_stats (a 40-byte uint8 tensor) to the host and decode it."""
    raw = bytes(stats_tensor.cpu().numpy().tobytes())
    return Stats.from_buffer_copy(raw[:C.sizeof(Stats)])


def new_stats(device="cuda:0") -> torch.Tensor:
    return torch.zeros(C.sizeof(Stats), dtype=torch.uint8, device=device)


class RouterBuffers:
    """All outputs of route_fwd for one context, allocated once."""

    def __init__(self, ctx: Context):
        p, dev, Cap = ctx.params, ctx.device, ctx.capacity
        self.logits = torch.empty(p.T, p.E, dtype=torch.float32, device=dev)
        self.scores = torch.empty(p.T, p.E, dtype=torch.float32, device=dev)
        self.expert_idx = torch.empty(p.T, p.k, dtype=torch.int32, device=dev)
        self.slot_idx = torch.empty(p.T, p.k, dtype=torch.int32, device=dev)
        self.gate_w = torch.empty(p.T, p.k, dtype=torch.float32, device=dev)
        self.slot_token = torch.empty(p.E, Cap, dtype=torch.int32, device=dev)
        self.expert_load = torch.empty(p.E, dtype=torch.int32, device=dev)
        self.stats = new_stats(dev)

    def args(self):
        return (self.logits, self.scores, self.expert_idx, self.slot_idx, self.gate_w, self.slot_token,
                self.expert_load, self.stats)

    def device_buffers(self, hidden, w_gate, expert_bias, xdisp) -> DeviceBuffers:
        d = DeviceBuffers()
        for name, t in (("hidden", hidden), ("w_gate", w_gate), ("expert_bias", expert_bias),
                        ("logits", self.logits), ("scores", self.scores), ("expert_idx", self.expert_idx),
                        ("slot_idx", self.slot_idx), ("gate_w", self.gate_w), ("slot_token", self.slot_token),
                        ("expert_load", self.expert_load), ("stats", self.stats), ("xdisp", xdisp)):
            setattr(d, name, t.data_ptr() if t is not None else None)
        return d
