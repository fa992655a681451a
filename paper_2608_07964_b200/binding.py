"""Thin ctypes binding of libeb.so: argument marshalling only.

Every step of the path (gating, scheduling, permutation, expert MLP, aggregation) runs in the
library's CUDA kernels; PyTorch is used here to own device memory and to supply the stream.
There is no CPU fallback: loading fails loudly when the library is missing.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import torch

from .build import LIB, build_library

EB_MAX_MB = 16
EB_MAX_D = 16
EB_META_LEN = 32
EB_HOST_SLOTS = 4

POLICY_MAXUTIL, POLICY_CUMUTIL, POLICY_DIFFPEAK, POLICY_ALL = 0, 1, 2, 3


class EbConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("L", "E", "K", "S", "H", "I", "D", "renorm_topk", "max_tokens")] + \
               [("expert_to_device", C.POINTER(C.c_int32))]


class EbBatch(C.Structure):
    _fields_ = [("n_mb", C.c_int32), ("tok_off", C.POINTER(C.c_int32)), ("layer", C.POINTER(C.c_int32)),
                ("pool_mask", C.c_uint32)]


class EbSchedResult(C.Structure):
    _fields_ = [("run_mask", C.c_uint32), ("defer_mask", C.c_uint32), ("n_run", C.c_int32), ("status", C.c_int32),
                ("joint_load", C.c_int32 * EB_MAX_D), ("util_num", C.c_int64), ("util_den", C.c_int64)]


class EbStepBuffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("logits", "x", "topk_idx", "topk_w", "mb_load", "mb_cnt", "sched",
                                          "group_off", "group_w", "row_src", "pos", "xp", "yp", "step_meta", "out",
                                          "residual")]


SYMBOLS = ["eb_create", "eb_destroy", "eb_bind_weights", "eb_workspace_bytes", "eb_set_workspace",
           "eb_rows_capacity", "eb_groups_capacity", "eb_route", "eb_schedule", "eb_permute",
           "eb_expert_ffn_grouped", "eb_expert_ffn_device", "eb_combine", "eb_combine_residual", "eb_step", "eb_step_host",
           "eb_step_host_submit", "eb_step_host_wait",
           "eb_permute_noalloc", "eb_selftest_bounded_wait", "eb_check_permutation", "eb_check_workspace_guards",
           "eb_device_status", "eb_num_kernels", "eb_kernel_name", "eb_set_timing", "eb_kernel_ms",
           "eb_launch_count", "eb_status_string", "eb_last_error"]

_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads libeb.so (building it first if its sources are newer); raises if unavailable."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB
    if path is None:
        try:
            build_library()
        except Exception as exc:  # nvcc missing on the box: use the shipped binary if there is one
            if not os.path.exists(p):
                raise RuntimeError(f"libeb.so is missing and could not be built: {exc}") from exc
    lib = C.CDLL(p)
    vp, i32, u32 = C.c_void_p, C.c_int32, C.c_uint32
    lib.eb_create.argtypes = [C.POINTER(EbConfig), C.POINTER(vp)]
    lib.eb_destroy.argtypes = [vp]
    lib.eb_bind_weights.argtypes = [vp, vp, vp, vp]
    lib.eb_workspace_bytes.argtypes = [vp]
    lib.eb_workspace_bytes.restype = C.c_size_t
    lib.eb_set_workspace.argtypes = [vp, vp, C.c_size_t]
    lib.eb_rows_capacity.argtypes = [vp]
    lib.eb_groups_capacity.argtypes = [vp]
    lib.eb_route.argtypes = [vp, vp, C.POINTER(EbBatch), u32, vp, vp, vp, vp, vp]
    lib.eb_schedule.argtypes = [vp, vp, C.POINTER(EbBatch), i32, i32, vp, vp, vp]
    lib.eb_permute.argtypes = [vp, vp, C.POINTER(EbBatch), vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.eb_expert_ffn_grouped.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.eb_expert_ffn_device.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32]
    lib.eb_combine.argtypes = [vp, vp, C.POINTER(EbBatch), vp, vp, vp, vp, vp]
    lib.eb_step.argtypes = [vp, vp, C.POINTER(EbBatch), u32, i32, i32, C.POINTER(EbStepBuffers)]
    lib.eb_combine_residual.argtypes = [vp, vp, C.POINTER(EbBatch), vp, vp, vp, vp, vp, vp]
    lib.eb_step_host.argtypes = [vp, vp, C.POINTER(EbBatch), u32, i32, i32, C.POINTER(EbStepBuffers), vp, vp, vp, vp]
    lib.eb_step_host_submit.argtypes = [vp, vp, C.POINTER(EbBatch), u32, i32, i32, C.POINTER(EbStepBuffers), vp, vp, vp, vp, i32]
    lib.eb_step_host_wait.argtypes = [vp, i32]
    lib.eb_permute_noalloc.argtypes = [C.POINTER(EbConfig), vp, C.POINTER(EbBatch), vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                       C.c_char_p, C.c_size_t]
    lib.eb_check_permutation.argtypes = [vp, vp, C.POINTER(EbBatch), vp, vp, vp, vp, vp, vp, vp, C.POINTER(i32)]
    lib.eb_check_workspace_guards.argtypes = [vp, vp, C.POINTER(i32)]
    lib.eb_selftest_bounded_wait.argtypes = [vp, vp, C.c_int64, C.POINTER(i32)]
    lib.eb_device_status.argtypes = [vp, C.POINTER(i32)]
    lib.eb_num_kernels.argtypes = []
    lib.eb_kernel_name.argtypes = [i32]
    lib.eb_kernel_name.restype = C.c_char_p
    lib.eb_set_timing.argtypes = [vp, i32]
    lib.eb_kernel_ms.argtypes = [vp, C.POINTER(C.c_float)]
    lib.eb_launch_count.argtypes = []
    lib.eb_launch_count.restype = C.c_uint64
    lib.eb_status_string.argtypes = [i32]
    lib.eb_status_string.restype = C.c_char_p
    lib.eb_last_error.argtypes = [vp]
    lib.eb_last_error.restype = C.c_char_p
    for name in SYMBOLS:
        if getattr(lib, name).restype is C.c_int:
            getattr(lib, name).restype = C.c_int32
    if path is None:
        _lib = lib
    return lib


class EbError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"eb error {code}: {msg}")
        self.code = code


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Batch:
    """Host-side description of the packed micro-batches of one call (kept alive for ctypes)."""

    def __init__(self, tok_off: Sequence[int], layers: Sequence[int], pool_mask: Optional[int] = None):
        n = len(layers)
        assert len(tok_off) == n + 1
        self.n_mb = n
        self.tok_off = list(tok_off)
        self.layers = list(layers)
        self._tok = (C.c_int32 * (n + 1))(*tok_off)
        self._lay = (C.c_int32 * max(n, 1))(*layers)
        self.pool_mask = ((1 << n) - 1) if pool_mask is None else pool_mask
        self.c = EbBatch(n, self._tok, self._lay, self.pool_mask)

    @property
    def n_tok(self) -> int:
        return self.tok_off[-1]


class MoEStep:
    """Owns an eb context plus the device buffers of one step (allocated with PyTorch)."""

    def __init__(self, L, E, K, S, H, I, D, expert_to_device: Sequence[int], max_tokens: int,
                 renorm_topk: int = 1, device: str = "cuda:0", lib_path: Optional[str] = None):
        self.lib = load_library(lib_path)
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.L, self.E, self.K, self.S, self.H, self.I, self.D = L, E, K, S, H, I, D
        self.max_tokens = max_tokens
        self._e2d = (C.c_int32 * E)(*expert_to_device)
        cfg = EbConfig(L, E, K, S, H, I, D, renorm_topk, max_tokens, self._e2d)
        h = C.c_void_p()
        self._check(self.lib.eb_create(C.byref(cfg), C.byref(h)), ctx=None)
        self.ctx = h
        self.rows_cap = self.lib.eb_rows_capacity(self.ctx)
        self.groups_cap = self.lib.eb_groups_capacity(self.ctx)
        nbytes = self.lib.eb_workspace_bytes(self.ctx)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.dev)
        self._check(self.lib.eb_set_workspace(self.ctx, self.workspace.data_ptr(), nbytes))
        i32, f32, bf = torch.int32, torch.float32, torch.bfloat16
        mk = lambda shape, dt: torch.empty(shape, dtype=dt, device=self.dev)
        self.logits = mk((max_tokens, E), f32)
        self.x = mk((max_tokens, H), bf)
        self.topk_idx = mk((max_tokens, K), i32)
        self.topk_w = mk((max_tokens, K), f32)
        self.mb_load = torch.zeros((EB_MAX_MB, D), dtype=i32, device=self.dev)
        self.mb_cnt = torch.zeros((EB_MAX_MB, E), dtype=i32, device=self.dev)
        self.sched = torch.zeros(C.sizeof(EbSchedResult), dtype=torch.uint8, device=self.dev)
        self.group_off = mk((self.groups_cap + 1,), i32)
        self.group_w = mk((self.groups_cap,), i32)
        self.row_src = mk((self.rows_cap,), i32)
        self.pos = mk((max_tokens, K + S), i32)
        self.xp = mk((self.rows_cap, H), bf)
        self.yp = mk((self.rows_cap, H), bf)
        self.step_meta = torch.zeros(EB_META_LEN, dtype=i32, device=self.dev)
        self.out = mk((max_tokens, H), bf)
        self.bufs = EbStepBuffers(*[t.data_ptr() for t in (
            self.logits, self.x, self.topk_idx, self.topk_w, self.mb_load, self.mb_cnt, self.sched, self.group_off,
            self.group_w, self.row_src, self.pos, self.xp, self.yp, self.step_meta, self.out)], None)
        # the same buffers with the hidden states updated in place: out = x + MoE(x) (Section 2.1)
        self.bufs_inplace = EbStepBuffers(*[t.data_ptr() for t in (
            self.logits, self.x, self.topk_idx, self.topk_w, self.mb_load, self.mb_cnt, self.sched, self.group_off,
            self.group_w, self.row_src, self.pos, self.xp, self.yp, self.step_meta, self.x)], self.x.data_ptr())
        self._weights = None

    # -- helpers -------------------------------------------------------------------------------
    def _check(self, code: int, ctx="self"):
        if code != 0:
            detail = ""
            if ctx is not None and getattr(self, "ctx", None):
                detail = self.lib.eb_last_error(self.ctx).decode()
            raise EbError(code, self.lib.eb_status_string(code).decode() + (": " + detail if detail else ""))

    def close(self):
        if getattr(self, "ctx", None):
            torch.cuda.synchronize(self.dev)
            self.lib.eb_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def bind_weights(self, w_gate: torch.Tensor, w_up: torch.Tensor, w_down: torch.Tensor):
        for w in (w_gate, w_up, w_down):
            assert w.is_cuda and w.dtype == torch.bfloat16 and w.is_contiguous()
        assert tuple(w_gate.shape) == (self.L, self.E + self.S, self.I, self.H) == tuple(w_up.shape)
        assert tuple(w_down.shape) == (self.L, self.E + self.S, self.H, self.I)
        self._weights = (w_gate, w_up, w_down)
        self._check(self.lib.eb_bind_weights(self.ctx, w_gate.data_ptr(), w_up.data_ptr(), w_down.data_ptr()))

    # -- the five calls ------------------------------------------------------------------------
    def eb_route(self, batch: Batch, route_mask: Optional[int] = None, logits: Optional[torch.Tensor] = None):
        lg = self.logits if logits is None else logits
        rm = ((1 << batch.n_mb) - 1) if route_mask is None else route_mask
        self._check(self.lib.eb_route(self.ctx, _stream(), C.byref(batch.c), rm, lg.data_ptr(), self.topk_idx.data_ptr(),
                                      self.topk_w.data_ptr(), self.mb_load.data_ptr(), self.mb_cnt.data_ptr()))

    def eb_schedule(self, batch: Batch, m: int, policy: int = POLICY_MAXUTIL, to_host: bool = False,
                    mb_load: Optional[torch.Tensor] = None) -> Optional[Dict]:
        h = EbSchedResult() if to_host else None
        ld = self.mb_load if mb_load is None else mb_load
        self._check(self.lib.eb_schedule(self.ctx, _stream(), C.byref(batch.c), m, policy, ld.data_ptr(),
                                         self.sched.data_ptr(), C.addressof(h) if to_host else None))
        return _sched_dict(h, self.D) if to_host else None

    def eb_permute(self, batch: Batch, x: Optional[torch.Tensor] = None):
        xx = self.x if x is None else x
        self._check(self.lib.eb_permute(self.ctx, _stream(), C.byref(batch.c), self.sched.data_ptr(), xx.data_ptr(),
                                        self.topk_idx.data_ptr(), self.group_off.data_ptr(), self.group_w.data_ptr(),
                                        self.row_src.data_ptr(), self.pos.data_ptr(), self.xp.data_ptr(),
                                        self.step_meta.data_ptr()))

    def eb_expert_ffn_grouped(self, device: Optional[int] = None):
        if device is None:
            self._check(self.lib.eb_expert_ffn_grouped(self.ctx, _stream(), self.xp.data_ptr(), self.group_off.data_ptr(),
                                                       self.group_w.data_ptr(), self.step_meta.data_ptr(), self.yp.data_ptr()))
        else:
            self._check(self.lib.eb_expert_ffn_device(self.ctx, _stream(), self.xp.data_ptr(), self.group_off.data_ptr(),
                                                      self.group_w.data_ptr(), self.step_meta.data_ptr(), self.yp.data_ptr(),
                                                      device))

    def eb_combine(self, batch: Batch, out: Optional[torch.Tensor] = None, residual: Optional[torch.Tensor] = None,
                   yp: Optional[torch.Tensor] = None):
        o = self.out if out is None else out
        y = self.yp if yp is None else yp
        if residual is None:
            self._check(self.lib.eb_combine(self.ctx, _stream(), C.byref(batch.c), self.sched.data_ptr(), y.data_ptr(),
                                            self.pos.data_ptr(), self.topk_w.data_ptr(), o.data_ptr()))
        else:
            self._check(self.lib.eb_combine_residual(self.ctx, _stream(), C.byref(batch.c), self.sched.data_ptr(),
                                                     y.data_ptr(), self.pos.data_ptr(), self.topk_w.data_ptr(),
                                                     residual.data_ptr(), o.data_ptr()))

    # -- whole step ----------------------------------------------------------------------------
    def eb_step(self, batch: Batch, m: int, policy: int = POLICY_MAXUTIL, route_mask: Optional[int] = None,
                in_place: bool = False):
        """The five calls back to back.  With `in_place` the hidden states self.x take x + MoE(x) for the chosen
        micro-batches (the aggregation adds the residual and writes over x); otherwise the MoE output goes to self.out."""
        rm = ((1 << batch.n_mb) - 1) if route_mask is None else route_mask
        bufs = self.bufs_inplace if in_place else self.bufs
        self._check(self.lib.eb_step(self.ctx, _stream(), C.byref(batch.c), rm, m, policy, C.byref(bufs)))

    def eb_step_host(self, batch: Batch, m: int, h_logits: torch.Tensor, h_x: torch.Tensor, h_out: torch.Tensor,
                     policy: int = POLICY_MAXUTIL, route_mask: Optional[int] = None) -> Dict:
        rm = ((1 << batch.n_mb) - 1) if route_mask is None else route_mask
        assert not h_logits.is_cuda and not h_x.is_cuda and not h_out.is_cuda
        if not hasattr(self, "_h_res"):
            self._h_res = EbSchedResult()     # one host result slot, so repeated calls have identical arguments
        h = self._h_res
        self._check(self.lib.eb_step_host(self.ctx, _stream(), C.byref(batch.c), rm, m, policy, C.byref(self.bufs),
                                          h_logits.data_ptr(), h_x.data_ptr(), h_out.data_ptr(), C.addressof(h)))
        return _sched_dict(h, self.D)

    def _slot_buffers(self, slot: int):
        """Per-slot buffers of the pipelined host path: (eb_step_buffers, pinned host result, device tensors).
        Inputs, schedule result and output are per slot; everything else is shared (the kernels of different
        slots run one after the other)."""
        if not hasattr(self, "_slots"):
            self._slots = {}
        if slot not in self._slots:
            f32, bf = torch.float32, torch.bfloat16
            mk = lambda shape, dt: torch.empty(shape, dtype=dt, device=self.dev)
            logits, x = mk((self.max_tokens, self.E), f32), mk((self.max_tokens, self.H), bf)
            sched = torch.zeros(C.sizeof(EbSchedResult), dtype=torch.uint8, device=self.dev)
            out = mk((self.max_tokens, self.H), bf)
            bufs = EbStepBuffers(*[t.data_ptr() for t in (
                logits, x, self.topk_idx, self.topk_w, self.mb_load, self.mb_cnt, sched, self.group_off,
                self.group_w, self.row_src, self.pos, self.xp, self.yp, self.step_meta, out)], None)
            h_res = torch.zeros(C.sizeof(EbSchedResult), dtype=torch.uint8).pin_memory()   # pinned: the copy back is asynchronous
            self._slots[slot] = (bufs, h_res, (logits, x, sched, out))
        return self._slots[slot]

    def step_host_submit(self, slot: int, batch: Batch, m: int, h_logits: torch.Tensor, h_x: torch.Tensor,
                         h_out: torch.Tensor, policy: int = POLICY_MAXUTIL, route_mask: Optional[int] = None):
        """Enqueues one host-to-host step on `slot` and returns; `step_host_wait(slot)` completes it."""
        rm = ((1 << batch.n_mb) - 1) if route_mask is None else route_mask
        assert not h_logits.is_cuda and not h_x.is_cuda and not h_out.is_cuda
        bufs, h_res, _ = self._slot_buffers(slot)
        self._check(self.lib.eb_step_host_submit(self.ctx, _stream(), C.byref(batch.c), rm, m, policy, C.byref(bufs),
                                                 h_logits.data_ptr(), h_x.data_ptr(), h_out.data_ptr(),
                                                 h_res.data_ptr(), slot))

    def step_host_wait(self, slot: int) -> Dict:
        self._check(self.lib.eb_step_host_wait(self.ctx, slot))
        h_res = self._slot_buffers(slot)[1]
        return _sched_dict(EbSchedResult.from_address(h_res.data_ptr()), self.D)

    # -- results and status --------------------------------------------------------------------
    def sched_result(self) -> Dict:
        raw = self.sched.cpu().numpy().tobytes()
        return _sched_dict(EbSchedResult.from_buffer_copy(raw), self.D)

    def meta(self) -> Dict:
        mvals = self.step_meta.cpu().tolist()
        return dict(rows=mvals[0], groups=mvals[1], active_layers=mvals[2], dev_group_off=mvals[3:3 + self.D + 1])

    def device_status(self) -> int:
        v = C.c_int32(0)
        self._check(self.lib.eb_device_status(self.ctx, C.byref(v)))
        return v.value

    def check_permutation(self, batch: Batch) -> int:
        """Number of inconsistencies the device-side checker finds in the tables of the last eb_permute."""
        v = C.c_int32(-1)
        self._check(self.lib.eb_check_permutation(self.ctx, _stream(), C.byref(batch.c), self.sched.data_ptr(),
                                                  self.topk_idx.data_ptr(), self.group_off.data_ptr(),
                                                  self.group_w.data_ptr(), self.row_src.data_ptr(), self.pos.data_ptr(),
                                                  self.step_meta.data_ptr(), C.byref(v)))
        return v.value

    def check_workspace_guards(self) -> int:
        """Guard bytes between the workspace regions that no longer hold their pattern (0 = intact)."""
        v = C.c_int32(-1)
        self._check(self.lib.eb_check_workspace_guards(self.ctx, _stream(), C.byref(v)))
        return v.value

    def selftest_bounded_wait(self, limit_cycles: int = 2_000_000) -> int:
        v = C.c_int32(-1)
        self._check(self.lib.eb_selftest_bounded_wait(self.ctx, _stream(), limit_cycles, C.byref(v)))
        return v.value

    def set_timing(self, on: bool):
        self._check(self.lib.eb_set_timing(self.ctx, 1 if on else 0))

    def kernel_ms(self) -> Dict[str, float]:
        n = self.lib.eb_num_kernels()
        arr = (C.c_float * n)()
        self._check(self.lib.eb_kernel_ms(self.ctx, arr))
        return {self.lib.eb_kernel_name(i).decode(): arr[i] for i in range(n) if arr[i] >= 0}


def permute_noalloc(L, E, K, S, H, D, expert_to_device: Sequence[int], batch: Batch, sched: torch.Tensor,
                    x: torch.Tensor, topk_idx: torch.Tensor, group_off: torch.Tensor, group_w: torch.Tensor,
                    row_src: torch.Tensor, pos: torch.Tensor, xp: torch.Tensor, step_meta: torch.Tensor) -> None:
    """eb_permute_noalloc: the dispatch step for callers that may not allocate device memory.

    No context and no workspace: the library's built-in static scratch is used, which limits the
    call to 4096 packed tokens.  All tensors are caller-owned device buffers."""
    lib = load_library()
    e2d = (C.c_int32 * E)(*expert_to_device)
    cfg = EbConfig(L, E, K, S, H, 8, D, 1, batch.n_tok, e2d)
    err = C.create_string_buffer(256)
    code = lib.eb_permute_noalloc(C.byref(cfg), _stream(), C.byref(batch.c), sched.data_ptr(), x.data_ptr(),
                                  topk_idx.data_ptr(), group_off.data_ptr(), group_w.data_ptr(), row_src.data_ptr(),
                                  pos.data_ptr(), xp.data_ptr(), step_meta.data_ptr(), err, 256)
    if code != 0:
        raise EbError(code, lib.eb_status_string(code).decode() + ": " + err.value.decode())


def launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(load_library().eb_launch_count())


def _sched_dict(h: EbSchedResult, D: int) -> Dict:
    return dict(run_mask=h.run_mask, defer_mask=h.defer_mask, n_run=h.n_run, status=h.status,
                joint_load=list(h.joint_load)[:D], util_num=h.util_num, util_den=h.util_den)


def from_workload(wl, device: str = "cuda:0", max_tokens: Optional[int] = None) -> MoEStep:
    """Context + buffers sized for a synthetic workload description (see synth.Workload)."""
    return MoEStep(wl.L, wl.E, wl.K, wl.S, wl.H, wl.I, wl.D, wl.expert_to_device(),
                   max_tokens or wl.T_tot, wl.renorm_topk, device)
