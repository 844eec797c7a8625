"""Thin ctypes binding over libsignmuon.so (argument marshalling only).

The functions below carry the names of the C ABI in include/signmuon.h.  `SignMuon`
bundles a context with the torch tensors that back its state and workspace; torch is
used for device memory and streams only.  There is no fallback: if the native library
is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsignmuon.so")

OK = 0
F32, BF16 = 0, 1
PARAM_MATRIX, PARAM_PLAIN = 0, 1
FLAG_KEEP_POLAR, FLAG_SIMT_GEMM, FLAG_GEMM_1CTA, FLAG_SIGN_AGREEMENT, FLAG_LP_GRAM_BF16 = 1, 2, 4, 16, 32
FLAG_NO_GRAM_SPACE = 64
STAGE_MOMENTUM, STAGE_NS, STAGE_VOTE, STAGE_LOCAL_POLAR, STAGE_ALL = 1, 2, 4, 8, 15
TAP_MOMENTUM, TAP_POLAR, TAP_VOTE_BITS, TAP_WORKER_BITS, TAP_NORM = 0, 1, 2, 3, 4

EXPORTS = [
    "signmuon_create", "signmuon_state_bytes", "signmuon_bind", "signmuon_step", "signmuon_run_stages",
    "signmuon_step_host", "signmuon_packed_payload", "signmuon_payload_buffer", "signmuon_vote_update",
    "signmuon_local_sign_sum", "signmuon_vote_update_from_sums", "signmuon_exchange_flags",
    "signmuon_set_payload_peers", "signmuon_payload_segment", "signmuon_debug_tap",
    "signmuon_status", "signmuon_launches_per_step", "signmuon_ns_launches_per_step", "signmuon_ns_flops_per_step", "signmuon_ns_executed_flops_per_step",
    "signmuon_power_start_size", "signmuon_power_start_segment", "signmuon_set_power_start",
    "signmuon_sign_agreement", "signmuon_set_wait_limit", "signmuon_selftest_wait_timeout",
    "signmuon_momentum_norm_noalloc", "signmuon_destroy", "signmuon_error_string",
]
NOALLOC_MAX_PARTIALS = 65536
ERR_TIMEOUT = -6
ERR_TOO_LARGE = -9
ERR_NO_MEMORY = -10


class ParamStruct(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("kind", C.c_int32),
                ("weight_dtype", C.c_int32), ("grad_dtype", C.c_int32)]


class ConfigStruct(C.Structure):
    _fields_ = [("num_params", C.c_int32), ("params", C.POINTER(ParamStruct)),
                ("num_workers", C.c_int32), ("momentum", C.c_float), ("lr", C.c_float),
                ("ns_steps", C.c_int32), ("local_polar", C.c_int32), ("weight_decay", C.c_float),
                ("eps", C.c_float), ("update_scale", C.c_int32), ("flags", C.c_int32),
                ("ns_scale", C.c_int32), ("power_iters", C.c_int32),
                ("worker_offset", C.c_int32), ("local_workers", C.c_int32), ("update_rule", C.c_int32)]


_lib = None


def load_library() -> C.CDLL:
    """Loads the native library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2605_16311_b200.build` "
                           "(there is no fallback implementation)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, f32, sz = C.c_void_p, C.c_int32, C.c_float, C.c_size_t
    lib.signmuon_create.argtypes = [C.POINTER(ConfigStruct), C.POINTER(vp)]
    lib.signmuon_state_bytes.argtypes = [vp, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)]
    lib.signmuon_bind.argtypes = [vp, vp, sz, vp, sz, vp, sz, C.c_int, vp]
    lib.signmuon_step.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), f32, vp]
    lib.signmuon_run_stages.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), f32, vp]
    lib.signmuon_step_host.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), f32, vp]
    lib.signmuon_packed_payload.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(sz), C.POINTER(sz)]
    lib.signmuon_payload_buffer.argtypes = [vp, C.POINTER(vp), C.POINTER(sz), C.POINTER(i32)]
    lib.signmuon_vote_update.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), f32, vp]
    lib.signmuon_exchange_flags.argtypes = [vp, C.POINTER(vp)]
    lib.signmuon_set_payload_peers.argtypes = [vp, i32, i32, i32, C.POINTER(vp), C.POINTER(vp)]
    lib.signmuon_local_sign_sum.argtypes = [vp, vp, sz, vp]
    lib.signmuon_vote_update_from_sums.argtypes = [vp, vp, sz, C.POINTER(vp), C.POINTER(vp), f32, vp]
    lib.signmuon_payload_segment.argtypes = [vp, i32, C.POINTER(sz), C.POINTER(sz)]
    lib.signmuon_debug_tap.argtypes = [vp, i32, i32, i32, C.POINTER(vp), C.POINTER(sz), C.POINTER(C.c_int64)]
    lib.signmuon_status.argtypes = [vp, vp]
    lib.signmuon_launches_per_step.argtypes = [vp, C.POINTER(i32)]
    lib.signmuon_ns_launches_per_step.argtypes = [vp, C.POINTER(i32), C.POINTER(i32)]
    lib.signmuon_ns_flops_per_step.argtypes = [vp, C.POINTER(C.c_double)]
    lib.signmuon_ns_executed_flops_per_step.argtypes = [vp, C.POINTER(C.c_double)]
    lib.signmuon_power_start_size.argtypes = [vp, C.POINTER(sz)]
    lib.signmuon_power_start_segment.argtypes = [vp, i32, C.POINTER(sz), C.POINTER(sz)]
    lib.signmuon_set_power_start.argtypes = [vp, vp, sz]
    lib.signmuon_sign_agreement.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), vp]
    lib.signmuon_set_wait_limit.argtypes = [vp, C.c_uint64]
    lib.signmuon_selftest_wait_timeout.argtypes = [vp, C.c_uint64, vp]
    lib.signmuon_momentum_norm_noalloc.argtypes = [vp, i32, vp, i32, vp, vp, vp, C.c_int64, C.c_int64, i32,
                                                   f32, f32, f32, vp]
    lib.signmuon_destroy.argtypes = [vp]
    lib.signmuon_destroy.restype = None
    lib.signmuon_error_string.argtypes = [C.c_int]
    lib.signmuon_error_string.restype = C.c_char_p
    for name in EXPORTS[:-2]:
        getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


class SignMuonError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().signmuon_error_string(code).decode()
        super().__init__(f"{where}: {msg} ({code})")


def _check(code: int, where: str):
    if code != OK:
        raise SignMuonError(code, where)


# ------------------------------------------------------------------------- C-ABI mirrors
def signmuon_create(params: Sequence[tuple], num_workers: int, momentum: float, lr: float, ns_steps: int,
                    local_polar: bool, weight_decay: float = 0.0, eps: float = 1e-12, update_scale: int = 0,
                    flags: int = 0, ns_scale: int = 0, power_iters: int = 2, worker_offset: int = 0,
                    local_workers: int = 0, update_rule: int = 0) -> int:
    """params: (rows, cols, kind, weight_dtype, grad_dtype) tuples. Returns the context handle."""
    lib = load_library()
    arr = (ParamStruct * max(len(params), 1))()
    for i, (r, c, k, wd, gd) in enumerate(params):
        arr[i] = ParamStruct(r, c, k, wd, gd)
    cfg = ConfigStruct(len(params), arr, num_workers, momentum, lr, ns_steps, int(local_polar), weight_decay,
                       eps, update_scale, flags, ns_scale, power_iters, worker_offset, local_workers, update_rule)
    out = C.c_void_p()
    _check(lib.signmuon_create(C.byref(cfg), C.byref(out)), "signmuon_create")
    return out.value


def signmuon_create_raw(cfg: Optional[ConfigStruct]):
    """Direct call for error-path tests: returns (code, handle)."""
    lib = load_library()
    out = C.c_void_p()
    code = lib.signmuon_create(C.byref(cfg) if cfg is not None else None, C.byref(out))
    return code, out.value


def signmuon_state_bytes(ctx: int):
    lib = load_library()
    a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(lib.signmuon_state_bytes(ctx, C.byref(a), C.byref(b), C.byref(c)), "signmuon_state_bytes")
    return a.value, b.value, c.value


def signmuon_bind(ctx: int, state_ptr: int, state_bytes: int, ws_ptr: int, ws_bytes: int, staging_ptr: int,
                  staging_bytes: int, zero_state: bool, stream: int):
    _check(load_library().signmuon_bind(ctx, state_ptr, state_bytes, ws_ptr, ws_bytes, staging_ptr or None,
                                        staging_bytes, int(zero_state), stream or None), "signmuon_bind")


def _ptr_array(ptrs: Sequence[int]):
    arr = (C.c_void_p * len(ptrs))()
    for i, p in enumerate(ptrs):
        arr[i] = p
    return arr


def signmuon_step(ctx: int, weight_ptrs, grad_ptrs, lr: float, stream: int):
    _check(load_library().signmuon_step(ctx, weight_ptrs, grad_ptrs, lr, stream or None), "signmuon_step")


def signmuon_run_stages(ctx: int, mask: int, weight_ptrs, grad_ptrs, lr: float, stream: int):
    _check(load_library().signmuon_run_stages(ctx, mask, weight_ptrs, grad_ptrs, lr, stream or None),
           "signmuon_run_stages")


def signmuon_step_host(ctx: int, weight_ptrs, grad_ptrs, lr: float, stream: int):
    _check(load_library().signmuon_step_host(ctx, weight_ptrs, grad_ptrs, lr, stream or None), "signmuon_step_host")


def signmuon_packed_payload(ctx: int, worker: int, want_ptr: bool = True):
    lib = load_library()
    p, b, e = C.c_void_p(), C.c_size_t(), C.c_size_t()
    _check(lib.signmuon_packed_payload(ctx, worker, C.byref(p) if want_ptr else None, C.byref(b), C.byref(e)),
           "signmuon_packed_payload")
    return p.value, b.value, e.value


def signmuon_payload_buffer(ctx: int, want_ptr: bool = True):
    """(device pointer of row 0, row pitch in bytes, rows) of the gathered payload buffer."""
    p, pitch, rows = C.c_void_p(), C.c_size_t(), C.c_int32()
    _check(load_library().signmuon_payload_buffer(ctx, C.byref(p) if want_ptr else None, C.byref(pitch), C.byref(rows)),
           "signmuon_payload_buffer")
    return p.value, pitch.value, rows.value


def signmuon_vote_update(ctx: int, payload_ptrs, weight_ptrs, grad_ptrs, lr: float, stream: int):
    _check(load_library().signmuon_vote_update(ctx, payload_ptrs, weight_ptrs, grad_ptrs, lr, stream or None),
           "signmuon_vote_update")


def signmuon_exchange_flags(ctx: int) -> int:
    p = C.c_void_p()
    _check(load_library().signmuon_exchange_flags(ctx, C.byref(p)), "signmuon_exchange_flags")
    return p.value


def signmuon_set_payload_peers(ctx: int, my_rank: int, num_ranks: int, peer_buffer_ptrs, peer_flag_ptrs):
    n = len(peer_buffer_ptrs)
    _check(load_library().signmuon_set_payload_peers(ctx, my_rank, num_ranks, n, _ptr_array(peer_buffer_ptrs) if n else None,
                                                     _ptr_array(peer_flag_ptrs) if n else None),
           "signmuon_set_payload_peers")


def signmuon_local_sign_sum(ctx: int, sums_ptr: int, nbytes: int, stream: int):
    _check(load_library().signmuon_local_sign_sum(ctx, sums_ptr, nbytes, stream or None), "signmuon_local_sign_sum")


def signmuon_vote_update_from_sums(ctx: int, sums_ptr: int, nbytes: int, weight_ptrs, grad_ptrs, lr: float, stream: int):
    _check(load_library().signmuon_vote_update_from_sums(ctx, sums_ptr, nbytes, weight_ptrs, grad_ptrs, lr,
                                                         stream or None), "signmuon_vote_update_from_sums")


def signmuon_payload_segment(ctx: int, param: int):
    lib = load_library()
    o, w = C.c_size_t(), C.c_size_t()
    _check(lib.signmuon_payload_segment(ctx, param, C.byref(o), C.byref(w)), "signmuon_payload_segment")
    return o.value, w.value


def signmuon_debug_tap(ctx: int, what: int, param: int, worker: int):
    lib = load_library()
    p, b, ld = C.c_void_p(), C.c_size_t(), C.c_int64()
    _check(lib.signmuon_debug_tap(ctx, what, param, worker, C.byref(p), C.byref(b), C.byref(ld)),
           "signmuon_debug_tap")
    return p.value, b.value, ld.value


def signmuon_status(ctx: int, stream: int) -> int:
    return load_library().signmuon_status(ctx, stream or None)


def signmuon_launches_per_step(ctx: int) -> int:
    n = C.c_int32()
    _check(load_library().signmuon_launches_per_step(ctx, C.byref(n)), "signmuon_launches_per_step")
    return n.value


def signmuon_ns_launches_per_step(ctx: int):
    g, ch = C.c_int32(), C.c_int32()
    _check(load_library().signmuon_ns_launches_per_step(ctx, C.byref(g), C.byref(ch)), "signmuon_ns_launches_per_step")
    return g.value, ch.value


def signmuon_ns_flops_per_step(ctx: int) -> float:
    f = C.c_double()
    _check(load_library().signmuon_ns_flops_per_step(ctx, C.byref(f)), "signmuon_ns_flops_per_step")
    return f.value


def signmuon_ns_executed_flops_per_step(ctx: int) -> float:
    f = C.c_double()
    _check(load_library().signmuon_ns_executed_flops_per_step(ctx, C.byref(f)), "signmuon_ns_executed_flops_per_step")
    return f.value


def signmuon_power_start_size(ctx: int) -> int:
    n = C.c_size_t()
    _check(load_library().signmuon_power_start_size(ctx, C.byref(n)), "signmuon_power_start_size")
    return n.value


def signmuon_power_start_segment(ctx: int, param: int):
    o, n = C.c_size_t(), C.c_size_t()
    _check(load_library().signmuon_power_start_segment(ctx, param, C.byref(o), C.byref(n)),
           "signmuon_power_start_segment")
    return o.value, n.value


def signmuon_set_power_start(ctx: int, ptr: int, floats: int):
    _check(load_library().signmuon_set_power_start(ctx, ptr, floats), "signmuon_set_power_start")


def signmuon_sign_agreement(ctx: int, num_workers: int, stream: int):
    """(per-worker counts of sign bits equal to the vote, entries per worker) of the last step."""
    agree = (C.c_uint64 * num_workers)()
    entries = C.c_uint64()
    _check(load_library().signmuon_sign_agreement(ctx, agree, C.byref(entries), stream or None),
           "signmuon_sign_agreement")
    return list(agree), entries.value


def signmuon_set_wait_limit(ctx: int, limit_ns: int):
    _check(load_library().signmuon_set_wait_limit(ctx, limit_ns), "signmuon_set_wait_limit")


def signmuon_selftest_wait_timeout(ctx: int, limit_ns: int, stream: int):
    _check(load_library().signmuon_selftest_wait_timeout(ctx, limit_ns, stream or None),
           "signmuon_selftest_wait_timeout")


def signmuon_momentum_norm_noalloc(grads_ptr: int, grad_dtype: int, weights_ptr: int, weight_dtype: int,
                                   momentum_ptr: int, operand_ptr: int, scales_ptr: int, rows: int, cols: int,
                                   num_workers: int, momentum: float, weight_decay: float, eps: float,
                                   stream: int) -> int:
    """Momentum + Frobenius-norm stage of one matrix with the library's built-in scratch: for callers
    that may not allocate device memory. Returns the C error code (0 = ok) instead of raising, so that
    the capacity refusal can be inspected."""
    return load_library().signmuon_momentum_norm_noalloc(
        grads_ptr, grad_dtype, weights_ptr or None, weight_dtype, momentum_ptr, operand_ptr, scales_ptr,
        rows, cols, num_workers, momentum, weight_decay, eps, stream or None)


def signmuon_destroy(ctx: int):
    load_library().signmuon_destroy(ctx)


# ------------------------------------------------------------------------- convenience wrapper
_DT = {"f32": F32, "bf16": BF16}
_KIND = {"matrix": PARAM_MATRIX, "plain": PARAM_PLAIN}
SCALES = {"fro": 0, "spectral": 1}
RULES = {"signmuon": 0, "muon": 1}
RULE_SIGNMUON, RULE_MUON = 0, 1


def _view_device(ptr: int, nbytes: int, dtype: torch.dtype, owner: torch.Tensor, base_ptr: int) -> torch.Tensor:
    """A tensor view of `nbytes` at device address `ptr`, which lies inside `owner` (uint8)."""
    off = ptr - base_ptr
    return owner[off: off + nbytes].view(dtype)


class SignMuon:
    """Owns a context plus the torch buffers behind it. `params` are workloads.Param-like objects
    (rows, cols, kind, dtype)."""

    def __init__(self, params, num_workers: int, momentum: float = 0.9, lr: float = 1e-3, ns_steps: int = 5,
                 local_polar: bool = False, weight_decay: float = 0.0, eps: float = 1e-12, update_scale: int = 0,
                 flags: int = 0, device: str = "cuda:0", host_staging: bool = False, ns_scale: str = "fro",
                 power_iters: int = 2, worker_offset: int = 0, local_workers: int = 0, update_rule: str = "signmuon"):
        self.params = list(params)
        self.num_workers = num_workers
        self.worker_offset = worker_offset if local_workers else 0
        self.local_workers = local_workers or num_workers      # workers this context computes
        self.sharded = self.local_workers < num_workers
        self.ns_steps = ns_steps
        self.device = torch.device(device)
        tuples = [(p.rows, p.cols, _KIND[p.kind], _DT[p.dtype], _DT[p.dtype]) for p in self.params]
        self.ctx = signmuon_create(tuples, num_workers, momentum, lr, ns_steps, local_polar, weight_decay, eps,
                                   update_scale, flags, SCALES[ns_scale], power_iters, worker_offset, local_workers,
                                   RULES[update_rule])
        self.state_bytes, self.workspace_bytes, self.staging_bytes = signmuon_state_bytes(self.ctx)
        with torch.cuda.device(self.device):
            self.state = torch.empty(self.state_bytes, dtype=torch.uint8, device=self.device)
            # over-allocate so the workspace can start on a 1024-byte boundary
            self._ws_raw = torch.empty(self.workspace_bytes + 1024, dtype=torch.uint8, device=self.device)
            off = (-self._ws_raw.data_ptr()) % 1024
            self.workspace = self._ws_raw[off: off + self.workspace_bytes]
            # (a sharded context stages host buffers itself, stage by stage: see step_host_sharded)
            self._host_stage = host_staging and self.sharded
            host_staging = host_staging and not self.sharded
            self.staging = (torch.empty(self.staging_bytes, dtype=torch.uint8, device=self.device)
                            if host_staging else None)
            stream = torch.cuda.current_stream(self.device).cuda_stream
            signmuon_bind(self.ctx, self.state.data_ptr(), self.state_bytes, self.workspace.data_ptr(),
                          self.workspace_bytes, self.staging.data_ptr() if host_staging else 0,
                          self.staging_bytes if host_staging else 0, True, stream)
        self._ptr_cache = None

    def rebind(self, zero_state: bool = True):
        """Binds the same buffers again (clears the device status word; optionally the momenta)."""
        with torch.cuda.device(self.device):
            stream = torch.cuda.current_stream(self.device).cuda_stream
            signmuon_bind(self.ctx, self.state.data_ptr(), self.state_bytes, self.workspace.data_ptr(),
                          self.workspace_bytes, self.staging.data_ptr() if self.staging is not None else 0,
                          self.staging_bytes if self.staging is not None else 0, zero_state, stream)

    def set_wait_limit(self, limit_ns: int):
        signmuon_set_wait_limit(self.ctx, limit_ns)

    def selftest_wait_timeout(self, limit_ns: int):
        signmuon_selftest_wait_timeout(self.ctx, limit_ns, torch.cuda.current_stream(self.device).cuda_stream)

    def close(self):
        if self.ctx:
            signmuon_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ptrs(self, weights: List[torch.Tensor], grads: List[torch.Tensor]):
        key = (tuple(w.data_ptr() for w in weights), tuple(g.data_ptr() for g in grads))
        if self._ptr_cache is None or self._ptr_cache[0] != key:
            self._ptr_cache = (key, _ptr_array(key[0]), _ptr_array(key[1]))
        return self._ptr_cache[1], self._ptr_cache[2]

    def step(self, weights, grads, lr: float = -1.0, stages: int = STAGE_ALL):
        wp, gp = self._ptrs(weights, grads)
        stream = torch.cuda.current_stream(self.device).cuda_stream
        if stages == STAGE_ALL:
            signmuon_step(self.ctx, wp, gp, lr, stream)
        else:
            signmuon_run_stages(self.ctx, stages, wp, gp, lr, stream)

    def step_host(self, host_weights, host_grads, lr: float = -1.0):
        wp, gp = self._ptrs(host_weights, host_grads)
        signmuon_step_host(self.ctx, wp, gp, lr, torch.cuda.current_stream(self.device).cuda_stream)

    # ---- worker sharding (Alg. 3 across GPUs): own workers' stages, exchange, shared stages
    def payload_rows(self) -> torch.Tensor:
        """int32 view [num_workers, pitch_words] of the gathered payload buffer (row m = worker m's payload)."""
        ptr, pitch, rows = signmuon_payload_buffer(self.ctx)
        flat = _view_device(ptr, pitch * rows, torch.int32, self.workspace, self.workspace.data_ptr())
        return flat.view(rows, pitch // 4)

    def exchange_payloads(self, dist_module, group=None):
        """All-gather of the packed words: every rank contributes the rows of its own workers."""
        from . import exchange
        exchange.all_gather_payload(self.payload_rows(), self.worker_offset, self.local_workers, dist_module, group)

    def set_payload_peers(self, my_rank: int, num_ranks: int, peers):
        """Fused exchange: `peers` are the SignMuon objects (or (payload buffer ptr, flags ptr) pairs of peer-mapped
        memory) whose payload buffers also receive every word this context packs."""
        pairs = [(signmuon_payload_buffer(p.ctx)[0], signmuon_exchange_flags(p.ctx)) if isinstance(p, SignMuon) else p
                 for p in peers]
        signmuon_set_payload_peers(self.ctx, my_rank, num_ranks, [a for a, _ in pairs], [b for _, b in pairs])

    def vote_update(self, weights, grads, lr: float = -1.0, payloads=None):
        """Vote, local polar step and update from the gathered payloads (payloads: optional list of num_workers
        device tensors or None entries; None = what the payload buffer already holds)."""
        wp, gp = self._ptrs(weights, grads)
        ptrs = [0] * self.num_workers if payloads is None else [0 if t is None else t.data_ptr() for t in payloads]
        signmuon_vote_update(self.ctx, _ptr_array(ptrs), wp, gp, lr, torch.cuda.current_stream(self.device).cuda_stream)

    def local_sign_sum(self, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """int8 sums of this context's own workers' signs, one per payload bit position (Alg. 2's all-reduce buffer)."""
        _, nbytes, _ = signmuon_packed_payload(self.ctx, self.worker_offset, want_ptr=False)
        if out is None:
            out = torch.empty(nbytes * 8, dtype=torch.int8, device=self.device)
        signmuon_local_sign_sum(self.ctx, out.data_ptr(), out.numel(), torch.cuda.current_stream(self.device).cuda_stream)
        return out

    def vote_update_from_sums(self, sums: torch.Tensor, weights, grads, lr: float = -1.0):
        wp, gp = self._ptrs(weights, grads)
        signmuon_vote_update_from_sums(self.ctx, sums.data_ptr(), sums.numel(), wp, gp, lr,
                                       torch.cuda.current_stream(self.device).cuda_stream)

    def step_sharded(self, weights, grads, lr: float, dist_module, group=None, int8_allreduce: bool = False):
        """One step of a sharded context: own workers' momentum + Newton-Schulz + pack, the exchange, then the
        shared vote / local polar / update (identical on every rank)."""
        self.step(weights, grads, lr, stages=STAGE_MOMENTUM | STAGE_NS)
        if int8_allreduce:
            from . import exchange
            sums = self.local_sign_sum(getattr(self, "_sums", None))
            self._sums = sums
            exchange.all_reduce_sign_sums(sums, dist_module, group)
            self.vote_update_from_sums(sums, weights, grads, lr)
        else:
            self.exchange_payloads(dist_module, group)
            self.step(weights, grads, lr, stages=STAGE_VOTE | STAGE_LOCAL_POLAR)

    def step_host_sharded(self, host_weights, host_grads, lr: float, dist_module, group=None):
        """step_sharded with host-resident weights and gradients: copies in, steps, copies the weights back."""
        if not hasattr(self, "_stage_w"):
            self._stage_w = [torch.empty_like(w, device=self.device) for w in host_weights]
            self._stage_g = [torch.empty_like(g, device=self.device) for g in host_grads]
        for dst, src in zip(self._stage_w, host_weights):
            dst.copy_(src, non_blocking=True)
        for dst, src in zip(self._stage_g, host_grads):
            dst.copy_(src, non_blocking=True)
        self.step_sharded(self._stage_w, self._stage_g, lr, dist_module, group)
        for dst, src in zip(host_weights, self._stage_w):
            dst.copy_(src, non_blocking=True)

    def status(self) -> int:
        return signmuon_status(self.ctx, torch.cuda.current_stream(self.device).cuda_stream)

    def payload(self, worker: int) -> torch.Tensor:
        """uint8 view of the bytes worker `worker` would transmit (valid until the next step)."""
        ptr, nbytes, _ = signmuon_packed_payload(self.ctx, worker)
        return _view_device(ptr, nbytes, torch.uint8, self.workspace, self.workspace.data_ptr())

    def tap(self, what: int, param: int, worker: int = 0) -> torch.Tensor:
        ptr, nbytes, ld = signmuon_debug_tap(self.ctx, what, param, worker)
        p = self.params[param]
        if what == TAP_MOMENTUM:
            return _view_device(ptr, nbytes, torch.float32, self.state, self.state.data_ptr()).view(p.rows, p.cols)
        base = self.workspace.data_ptr()
        if what == TAP_POLAR:
            return _view_device(ptr, nbytes, torch.bfloat16, self.workspace, base).view(p.rows, ld)[:, : p.cols]
        if what in (TAP_VOTE_BITS, TAP_WORKER_BITS):
            return _view_device(ptr, nbytes, torch.uint8, self.workspace, base)
        if what == TAP_NORM:
            return _view_device(ptr, nbytes, torch.float32, self.workspace, base)
        raise ValueError(what)

    def power_start_segment(self, param: int):
        """(offset, floats per worker) of a matrix parameter's start vectors inside the start-vector array."""
        return signmuon_power_start_segment(self.ctx, param)

    def sign_agreement(self):
        return signmuon_sign_agreement(self.ctx, self.num_workers, torch.cuda.current_stream(self.device).cuda_stream)

    @property
    def power_start_size(self) -> int:
        return signmuon_power_start_size(self.ctx)

    def set_power_start(self, vectors: torch.Tensor):
        """float32 device tensor of power_start_size floats: the sampled start vectors of Alg. 5; the caller keeps it alive."""
        assert vectors.dtype == torch.float32 and vectors.is_cuda and vectors.is_contiguous()
        self._power_start = vectors
        signmuon_set_power_start(self.ctx, vectors.data_ptr(), vectors.numel())

    @property
    def launches_per_step(self) -> int:
        return signmuon_launches_per_step(self.ctx)

    @property
    def ns_launches_per_step(self):
        """(grouped tensor-core product launches, on-chip chain launches) of the Newton-Schulz work of one step."""
        return signmuon_ns_launches_per_step(self.ctx)

    @property
    def ns_flops_per_step(self) -> float:
        return signmuon_ns_flops_per_step(self.ctx)

    @property
    def ns_executed_flops_per_step(self) -> float:
        return signmuon_ns_executed_flops_per_step(self.ctx)
