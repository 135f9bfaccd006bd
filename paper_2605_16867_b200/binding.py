"""ctypes binding with the same names as the C ABI (see include/goodserve.h).

Argument marshalling only: tensors are checked (device, dtype, contiguity) and their
addresses handed to the library.  PyTorch supplies device memory and streams, nothing else.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
GS_ROUTE_ACCUMULATE = 1


class DeviceStatus:
    BAD_INSTANCE = 1
    BAD_TYPE = 2
    BAD_VALUE = 4
    TIMEOUT = 8
    CAND_TRUNCATED = 16
    INTERNAL = 32


class GoodServeError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"libgoodserve error {code}: {message}")
        self.code = code


class _Instances(C.Structure):
    _fields_ = [("type_id", C.c_void_p), ("queued_prefill_tokens", C.c_void_p),
                ("decode_batch", C.c_void_p), ("free_kv_tokens", C.c_void_p),
                ("q_ema_ms", C.c_void_p), ("n_instances", C.c_int32)]


class _Types(C.Structure):
    _fields_ = [("prefill_ms_per_tok", C.c_void_p), ("tpot_a_ms", C.c_void_p),
                ("tpot_b_ms", C.c_void_p), ("n_types", C.c_int32)]


class _InstanceTable(C.Structure):
    _fields_ = [("q_ms", C.c_void_p), ("p_ms_per_tok", C.c_void_p), ("d_ms_per_tok", C.c_void_p),
                ("free_kv_tokens", C.c_void_p), ("n_instances", C.c_int32)]


class _InstancesMut(C.Structure):
    _fields_ = [("queued_prefill_tokens", C.c_void_p), ("decode_batch", C.c_void_p),
                ("free_kv_tokens", C.c_void_p), ("q_ema_ms", C.c_void_p),
                ("n_instances", C.c_int32)]


def library_path(counting: bool = False, checking: bool = False) -> str:
    name = "libgoodserve_count.so" if counting else "libgoodserve_debug.so" if checking else "libgoodserve.so"
    return os.path.join(_PKG, name)


_libs = {}


def _declare(lib):
    """Argument and result types of every entry point of include/goodserve.h."""
    vp, i32, i64, f32, u32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_uint
    lib.gs_create.argtypes = [C.POINTER(vp), C.c_int, C.c_int, C.c_int]
    lib.gs_destroy.argtypes = [vp]
    lib.gs_strerror.argtypes = [C.c_int]
    lib.gs_strerror.restype = C.c_char_p
    lib.gs_last_cuda_error.argtypes = [vp]
    lib.gs_device_status.argtypes = [vp, vp, C.POINTER(u32)]
    lib.gs_launch_count.argtypes = [vp]
    lib.gs_launch_count.restype = i64
    lib.gs_eval_counters.argtypes = [vp, vp, C.POINTER(C.c_uint64), C.c_int]
    lib.gs_eval_counters.restype = C.c_int
    route_args = [vp, vp, vp, vp, i64, C.POINTER(_Instances), C.POINTER(_Types), f32, vp, vp, vp, vp]
    lib.gs_route_batch.argtypes = route_args + [u32, vp]
    lib.gs_route_batch_host.argtypes = route_args + [vp]
    lib.gs_route_batch_host_deferred.argtypes = route_args + [vp]
    lib.gs_host_wait.argtypes = [vp, vp]
    lib.gs_route_batch_prefix.argtypes = [vp, vp, vp, vp, i64, vp, vp, C.c_int, i64, C.POINTER(_Instances),
                                          C.POINTER(_Types), f32, vp, vp, vp, vp, vp]
    lib.gs_route_batch_prefix.restype = C.c_int
    lib.gs_route_batch_direct.argtypes = [vp, vp, vp, vp, i64, C.POINTER(_InstanceTable), vp, vp, vp, vp, vp]
    lib.gs_route_batch_direct.restype = C.c_int
    lib.gs_ema_update.argtypes = [vp, f32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.gs_ema_update.restype = C.c_int
    lib.gs_route_sequential.argtypes = [vp, vp, vp, vp, i64, vp, C.POINTER(_InstancesMut), C.POINTER(_Types), f32,
                                        vp, vp, vp, vp, vp]
    lib.gs_route_sequential.restype = C.c_int
    lib.gs_advance_state.argtypes = [vp, C.POINTER(_InstancesMut), vp]
    risk_args = [vp, vp, vp, vp, vp, vp, i64, C.POINTER(_Instances), C.POINTER(_Types), vp, vp, i64, vp, vp]
    lib.gs_risk_scan.argtypes = risk_args
    lib.gs_risk_scan_host.argtypes = risk_args
    lib.gs_timing_enable.argtypes = [vp, C.c_int]
    lib.gs_timing_read.argtypes = [vp, C.c_int, C.POINTER(C.c_double), C.POINTER(i64)]
    lib.gs_reroute_candidates.argtypes = [vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, i64, C.POINTER(_Instances),
                                          C.POINTER(_Types), f32, vp, vp, vp, vp, vp]
    lib.gs_reroute_candidates.restype = C.c_int
    lib.gs_risk_scan_noalloc.argtypes = [vp, vp, vp, vp, vp, i64, C.POINTER(_Instances), C.POINTER(_Types),
                                         vp, vp, i64, vp, vp, vp]
    lib.gs_risk_scan_noalloc.restype = C.c_int
    for name in ("gs_timing_enable", "gs_timing_read", "gs_create", "gs_destroy", "gs_last_cuda_error", "gs_device_status", "gs_route_batch",
                 "gs_route_batch_host", "gs_route_batch_host_deferred", "gs_host_wait", "gs_advance_state", "gs_risk_scan", "gs_risk_scan_host"):
        getattr(lib, name).restype = C.c_int
    return lib


def load_library(build_if_missing: bool = True, counting: bool = False, checking: bool = False):
    """Loads libgoodserve.so (building it with nvcc first if it is absent or stale).
    Raises if that fails -- there is no other implementation to fall back to.
    ``counting=True`` loads the measuring build instead (-DGS_COUNT_EVALS: the work counters
    behind gs_eval_counters tick; many times slower, for benchmarks only); ``checking=True`` the
    build with table index checks compiled in (-DGS_DEBUG; GS_DEV_INTERNAL reports a failure)."""
    kind = "counting" if counting else "checking" if checking else "regular"
    if kind in _libs:
        return _libs[kind]
    path = library_path(counting, checking)
    if build_if_missing:
        from .build import build_library
        try:
            build_library(counting=counting, checking=checking)
        except Exception as exc:                      # nvcc missing on a box that has the .so
            if not os.path.exists(path):
                raise RuntimeError(f"{os.path.basename(path)} is missing and could not be built: {exc}") from exc
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found; run paper_2605_16867_b200/build.py")
    _libs[kind] = _declare(C.CDLL(path))
    return _libs[kind]


def _dev_ptr(t: Optional[torch.Tensor], dtype: torch.dtype, n: Optional[int], name: str, device) -> Optional[int]:
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name}: expected a CUDA tensor")
    if t.device != device:
        raise ValueError(f"{name}: tensor is on {t.device}, context is on {device}")
    if t.dtype != dtype or not t.is_contiguous() or t.dim() != 1:
        raise TypeError(f"{name}: expected a contiguous 1-D {dtype} tensor, got {t.dtype} {tuple(t.shape)}")
    if n is not None and t.numel() < n:
        raise ValueError(f"{name}: needs {n} elements, has {t.numel()}")
    return t.data_ptr()


def _host_ptr(a, dtype, n: Optional[int], name: str) -> Optional[int]:
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        if a.is_cuda or not a.is_contiguous():
            raise TypeError(f"{name}: expected a contiguous host tensor")
        if n is not None and a.numel() < n:
            raise ValueError(f"{name}: needs {n} elements, has {a.numel()}")
        return a.data_ptr()
    if not isinstance(a, np.ndarray) or a.dtype != dtype or not a.flags.c_contiguous:
        raise TypeError(f"{name}: expected a contiguous numpy array of {dtype}")
    if n is not None and a.size < n:
        raise ValueError(f"{name}: needs {n} elements, has {a.size}")
    return a.ctypes.data


@dataclass
class InstancePool:
    """Device-resident pool description: per-instance state (SoA) and the type table."""
    type_id: torch.Tensor
    queued_prefill_tokens: torch.Tensor
    decode_batch: torch.Tensor
    free_kv_tokens: torch.Tensor
    q_ema_ms: torch.Tensor
    prefill_ms_per_tok: torch.Tensor
    tpot_a_ms: torch.Tensor
    tpot_b_ms: torch.Tensor

    @property
    def n_instances(self) -> int:
        return int(self.type_id.numel())

    @property
    def n_types(self) -> int:
        return int(self.prefill_ms_per_tok.numel())

    @staticmethod
    def from_host(types, inst, device) -> "InstancePool":
        def up(a):
            return torch.from_numpy(np.ascontiguousarray(a)).to(device)
        return InstancePool(up(inst.type_id), up(inst.queued_prefill_tokens), up(inst.decode_batch),
                            up(inst.free_kv_tokens), up(inst.q_ema_ms), up(types.prefill_ms_per_tok),
                            up(types.tpot_a_ms), up(types.tpot_b_ms))


class GoodServe:
    """One library context (gs_create / gs_destroy) bound to a CUDA device."""

    def __init__(self, device: int = 0, max_instances: int = 1024, max_types: int = 16, counting: bool = False,
                 checking: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("GoodServe needs a CUDA device; there is no CPU implementation")
        self._lib = load_library(counting=counting, checking=checking)
        self.device = torch.device("cuda", device)
        torch.cuda.init()
        with torch.cuda.device(self.device):
            torch.zeros(1, device=self.device)          # make sure the primary context exists
        h = C.c_void_p()
        self._check(self._lib.gs_create(C.byref(h), device, max_instances, max_types))
        self._h = h
        self._deferred = None

    # -- plumbing ------------------------------------------------------------------------
    def _check(self, rc: int):
        if rc != 0:
            raise GoodServeError(rc, self._lib.gs_strerror(rc).decode())

    def _stream(self, stream) -> Optional[int]:
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        return s.cuda_stream or None

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.gs_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _pool_structs(self, pool: InstancePool):
        M, Tn, dev = pool.n_instances, pool.n_types, self.device
        i32, f32 = torch.int32, torch.float32
        inst = _Instances(_dev_ptr(pool.type_id, i32, M, "type_id", dev),
                          _dev_ptr(pool.queued_prefill_tokens, i32, M, "queued_prefill_tokens", dev),
                          _dev_ptr(pool.decode_batch, i32, M, "decode_batch", dev),
                          _dev_ptr(pool.free_kv_tokens, i32, M, "free_kv_tokens", dev),
                          _dev_ptr(pool.q_ema_ms, f32, M, "q_ema_ms", dev), M)
        types = _Types(_dev_ptr(pool.prefill_ms_per_tok, f32, Tn, "prefill_ms_per_tok", dev),
                       _dev_ptr(pool.tpot_a_ms, f32, Tn, "tpot_a_ms", dev),
                       _dev_ptr(pool.tpot_b_ms, f32, Tn, "tpot_b_ms", dev), Tn)
        return inst, types

    @staticmethod
    def _host_pool_structs(types, inst):
        M, Tn = int(inst.type_id.shape[0]), int(types.prefill_ms_per_tok.shape[0])
        hi = _Instances(_host_ptr(inst.type_id, np.int32, M, "type_id"),
                        _host_ptr(inst.queued_prefill_tokens, np.int32, M, "queued_prefill_tokens"),
                        _host_ptr(inst.decode_batch, np.int32, M, "decode_batch"),
                        _host_ptr(inst.free_kv_tokens, np.int32, M, "free_kv_tokens"),
                        _host_ptr(inst.q_ema_ms, np.float32, M, "q_ema_ms"), M)
        ht = _Types(_host_ptr(types.prefill_ms_per_tok, np.float32, Tn, "prefill_ms_per_tok"),
                    _host_ptr(types.tpot_a_ms, np.float32, Tn, "tpot_a_ms"),
                    _host_ptr(types.tpot_b_ms, np.float32, Tn, "tpot_b_ms"), Tn)
        return hi, ht

    # -- C ABI, same names ----------------------------------------------------------------
    def route_batch(self, prompt_len, pred_decode_len, slo_ms, pool: InstancePool, ema_alpha: float,
                    out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier=None,
                    accumulate: bool = False, n_requests: Optional[int] = None, stream=None):
        n = int(prompt_len.numel()) if n_requests is None else int(n_requests)
        dev, i32, f32 = self.device, torch.int32, torch.float32
        inst, types = self._pool_structs(pool)
        self._check(self._lib.gs_route_batch(
            self._h, _dev_ptr(prompt_len, i32, n, "prompt_len", dev),
            _dev_ptr(pred_decode_len, i32, n, "pred_decode_len", dev),
            _dev_ptr(slo_ms, f32, n, "slo_ms", dev), n, C.byref(inst), C.byref(types),
            float(ema_alpha), _dev_ptr(out_instance_idx, i32, n, "out_instance_idx", dev),
            _dev_ptr(out_est_e2e_ms, f32, n, "out_est_e2e_ms", dev),
            _dev_ptr(out_slack_ms, f32, n, "out_slack_ms", dev),
            _dev_ptr(out_tier, torch.uint8, n, "out_tier", dev),
            GS_ROUTE_ACCUMULATE if accumulate else 0, self._stream(stream)))

    def route_batch_prefix(self, prompt_len, pred_decode_len, slo_ms, prefix_inst, prefix_hit_len,
                           n_slots: int, slot_stride: int, pool: InstancePool, ema_alpha: float,
                           out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier=None,
                           n_requests: Optional[int] = None, stream=None):
        """``prefix_inst`` / ``prefix_hit_len``: 1-D int32 CUDA tensors of n_slots * slot_stride
        entries, slot k of request r at k * slot_stride + r."""
        n = int(prompt_len.numel()) if n_requests is None else int(n_requests)
        dev, i32, f32 = self.device, torch.int32, torch.float32
        inst, types = self._pool_structs(pool)
        n_hits = max(int(n_slots), 0) * int(slot_stride)
        self._check(self._lib.gs_route_batch_prefix(
            self._h, _dev_ptr(prompt_len, i32, n, "prompt_len", dev),
            _dev_ptr(pred_decode_len, i32, n, "pred_decode_len", dev),
            _dev_ptr(slo_ms, f32, n, "slo_ms", dev), n,
            _dev_ptr(prefix_inst, i32, n_hits, "prefix_inst", dev),
            _dev_ptr(prefix_hit_len, i32, n_hits, "prefix_hit_len", dev), int(n_slots), int(slot_stride),
            C.byref(inst), C.byref(types),
            float(ema_alpha), _dev_ptr(out_instance_idx, i32, n, "out_instance_idx", dev),
            _dev_ptr(out_est_e2e_ms, f32, n, "out_est_e2e_ms", dev),
            _dev_ptr(out_slack_ms, f32, n, "out_slack_ms", dev),
            _dev_ptr(out_tier, torch.uint8, n, "out_tier", dev), self._stream(stream)))

    def route_batch_direct(self, prompt_len, pred_decode_len, slo_ms, q_ms, p_ms_per_tok, d_ms_per_tok,
                           free_kv_tokens, out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier=None,
                           n_requests: Optional[int] = None, n_instances: Optional[int] = None, stream=None):
        """Routing round against per-instance coefficients given directly (CUDA tensors)."""
        n = int(prompt_len.numel()) if n_requests is None else int(n_requests)
        M = int(q_ms.numel()) if n_instances is None else int(n_instances)
        dev, i32, f32 = self.device, torch.int32, torch.float32
        table = _InstanceTable(_dev_ptr(q_ms, f32, M, "q_ms", dev), _dev_ptr(p_ms_per_tok, f32, M, "p_ms_per_tok", dev),
                               _dev_ptr(d_ms_per_tok, f32, M, "d_ms_per_tok", dev),
                               _dev_ptr(free_kv_tokens, i32, M, "free_kv_tokens", dev), M)
        self._check(self._lib.gs_route_batch_direct(
            self._h, _dev_ptr(prompt_len, i32, n, "prompt_len", dev),
            _dev_ptr(pred_decode_len, i32, n, "pred_decode_len", dev),
            _dev_ptr(slo_ms, f32, n, "slo_ms", dev), n, C.byref(table),
            _dev_ptr(out_instance_idx, i32, n, "out_instance_idx", dev),
            _dev_ptr(out_est_e2e_ms, f32, n, "out_est_e2e_ms", dev),
            _dev_ptr(out_slack_ms, f32, n, "out_slack_ms", dev),
            _dev_ptr(out_tier, torch.uint8, n, "out_tier", dev), self._stream(stream)))

    def ema_update(self, alpha: float, obs_q_ms, obs_p_ms_per_tok, obs_d_ms_per_tok, q_ms, p_ms_per_tok,
                   d_ms_per_tok, n_instances: Optional[int] = None, stream=None):
        """In-place EMA step of the coefficient columns; a ``None`` observation skips its column."""
        cols = [t for t in (q_ms, p_ms_per_tok, d_ms_per_tok, obs_q_ms, obs_p_ms_per_tok, obs_d_ms_per_tok) if t is not None]
        M = int(cols[0].numel()) if n_instances is None else int(n_instances)
        dev, f32 = self.device, torch.float32
        self._check(self._lib.gs_ema_update(
            self._h, float(alpha), M, _dev_ptr(obs_q_ms, f32, M, "obs_q_ms", dev),
            _dev_ptr(obs_p_ms_per_tok, f32, M, "obs_p_ms_per_tok", dev),
            _dev_ptr(obs_d_ms_per_tok, f32, M, "obs_d_ms_per_tok", dev), _dev_ptr(q_ms, f32, M, "q_ms", dev),
            _dev_ptr(p_ms_per_tok, f32, M, "p_ms_per_tok", dev), _dev_ptr(d_ms_per_tok, f32, M, "d_ms_per_tok", dev),
            self._stream(stream)))

    def route_sequential(self, prompt_len, pred_decode_len, slo_ms, pool: InstancePool, ema_alpha: float,
                         out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier=None,
                         n_requests: Optional[int] = None, stream=None):
        """One request at a time; ``pool``'s state tensors are advanced in place."""
        n = int(prompt_len.numel()) if n_requests is None else int(n_requests)
        M, dev, i32, f32 = pool.n_instances, self.device, torch.int32, torch.float32
        _, types = self._pool_structs(pool)
        mut = _InstancesMut(_dev_ptr(pool.queued_prefill_tokens, i32, M, "queued_prefill_tokens", dev),
                            _dev_ptr(pool.decode_batch, i32, M, "decode_batch", dev),
                            _dev_ptr(pool.free_kv_tokens, i32, M, "free_kv_tokens", dev),
                            _dev_ptr(pool.q_ema_ms, f32, M, "q_ema_ms", dev), M)
        self._check(self._lib.gs_route_sequential(
            self._h, _dev_ptr(prompt_len, i32, n, "prompt_len", dev),
            _dev_ptr(pred_decode_len, i32, n, "pred_decode_len", dev),
            _dev_ptr(slo_ms, f32, n, "slo_ms", dev), n, _dev_ptr(pool.type_id, i32, M, "type_id", dev),
            C.byref(mut), C.byref(types), float(ema_alpha),
            _dev_ptr(out_instance_idx, i32, n, "out_instance_idx", dev),
            _dev_ptr(out_est_e2e_ms, f32, n, "out_est_e2e_ms", dev),
            _dev_ptr(out_slack_ms, f32, n, "out_slack_ms", dev),
            _dev_ptr(out_tier, torch.uint8, n, "out_tier", dev), self._stream(stream)))

    def advance_state(self, pool: InstancePool, stream=None):
        M, dev, i32 = pool.n_instances, self.device, torch.int32
        mut = _InstancesMut(_dev_ptr(pool.queued_prefill_tokens, i32, M, "queued_prefill_tokens", dev),
                            _dev_ptr(pool.decode_batch, i32, M, "decode_batch", dev),
                            _dev_ptr(pool.free_kv_tokens, i32, M, "free_kv_tokens", dev),
                            _dev_ptr(pool.q_ema_ms, torch.float32, M, "q_ema_ms", dev), M)
        self._check(self._lib.gs_advance_state(self._h, C.byref(mut), self._stream(stream)))

    def risk_scan(self, assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms,
                  pool: InstancePool, out_flag_bits, out_cand_idx, out_cand_count,
                  cand_capacity: Optional[int] = None, n_active: Optional[int] = None, stream=None):
        n = int(assigned_inst.numel()) if n_active is None else int(n_active)
        cap = (0 if out_cand_idx is None else int(out_cand_idx.numel())) if cand_capacity is None else int(cand_capacity)
        dev, i32, f32 = self.device, torch.int32, torch.float32
        inst, types = self._pool_structs(pool)
        self._check(self._lib.gs_risk_scan(
            self._h, _dev_ptr(assigned_inst, i32, n, "assigned_inst", dev),
            _dev_ptr(generated_tokens, i32, n, "generated_tokens", dev),
            _dev_ptr(pred_len, i32, n, "pred_len", dev),
            _dev_ptr(elapsed_ms, f32, n, "elapsed_ms", dev), _dev_ptr(slo_ms, f32, n, "slo_ms", dev), n,
            C.byref(inst), C.byref(types),
            _dev_ptr(out_flag_bits, i32, (n + 31) // 32, "out_flag_bits", dev),
            _dev_ptr(out_cand_idx, i32, cap, "out_cand_idx", dev), cap,
            _dev_ptr(out_cand_count, torch.int64, 1, "out_cand_count", dev), self._stream(stream)))

    def reroute_candidates(self, cand_idx, cand_count, assigned_inst, generated_tokens, pred_len, elapsed_ms,
                           slo_ms, prompt_len, pool: InstancePool, ema_alpha: float,
                           out_new_instance, out_est_ms, out_slack_ms, out_tier=None,
                           cand_capacity: Optional[int] = None, stream=None):
        """gs_reroute_candidates: cand_idx / cand_count are risk_scan's device outputs."""
        cap = int(cand_idx.numel()) if cand_capacity is None else int(cand_capacity)
        n = int(assigned_inst.numel())
        dev, i32, f32 = self.device, torch.int32, torch.float32
        inst, types = self._pool_structs(pool)
        self._check(self._lib.gs_reroute_candidates(
            self._h, _dev_ptr(cand_idx, i32, cap, "cand_idx", dev),
            _dev_ptr(cand_count, torch.int64, 1, "cand_count", dev), cap,
            _dev_ptr(assigned_inst, i32, n, "assigned_inst", dev),
            _dev_ptr(generated_tokens, i32, n, "generated_tokens", dev),
            _dev_ptr(pred_len, i32, n, "pred_len", dev), _dev_ptr(elapsed_ms, f32, n, "elapsed_ms", dev),
            _dev_ptr(slo_ms, f32, n, "slo_ms", dev), _dev_ptr(prompt_len, i32, n, "prompt_len", dev), n,
            C.byref(inst), C.byref(types), float(ema_alpha),
            _dev_ptr(out_new_instance, i32, cap, "out_new_instance", dev),
            _dev_ptr(out_est_ms, f32, cap, "out_est_ms", dev),
            _dev_ptr(out_slack_ms, f32, cap, "out_slack_ms", dev),
            _dev_ptr(out_tier, torch.uint8, cap, "out_tier", dev), self._stream(stream)))

    def route_batch_host(self, prompt_len, pred_decode_len, slo_ms, types, inst, ema_alpha: float,
                         out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier=None, stream=None,
                         wait: bool = True):
        """Host-buffer variant: numpy arrays or (pinned) host tensors in and out.  With
        ``wait=False`` the call returns once everything is enqueued (gs_route_batch_host_deferred):
        the outputs are valid after ``host_wait()`` or the next host-buffer call has returned."""
        n = int(prompt_len.shape[0])
        hi, ht = self._host_pool_structs(types, inst)
        fn = self._lib.gs_route_batch_host if wait else self._lib.gs_route_batch_host_deferred
        if not wait:        # what the enqueued copies read and write stays referenced until the wait
            self._deferred = (prompt_len, pred_decode_len, slo_ms, types, inst, hi, ht,
                              out_instance_idx, out_est_e2e_ms, out_slack_ms, out_tier)
        self._check(fn(
            self._h, _host_ptr(prompt_len, np.int32, n, "prompt_len"),
            _host_ptr(pred_decode_len, np.int32, n, "pred_decode_len"),
            _host_ptr(slo_ms, np.float32, n, "slo_ms"), n, C.byref(hi), C.byref(ht), float(ema_alpha),
            _host_ptr(out_instance_idx, np.int32, n, "out_instance_idx"),
            _host_ptr(out_est_e2e_ms, np.float32, n, "out_est_e2e_ms"),
            _host_ptr(out_slack_ms, np.float32, n, "out_slack_ms"),
            _host_ptr(out_tier, np.uint8, n, "out_tier"), self._stream(stream)))

    def host_wait(self, stream=None):
        """Waits for what the host-buffer calls have enqueued (gs_host_wait)."""
        self._check(self._lib.gs_host_wait(self._h, self._stream(stream)))
        self._deferred = None

    def risk_scan_host(self, assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms, types, inst,
                       out_flag_bits, out_cand_idx, stream=None) -> int:
        """Host-buffer variant; returns the true number of flagged requests."""
        n = int(assigned_inst.shape[0])
        cap = 0 if out_cand_idx is None else int(out_cand_idx.shape[0])
        hi, ht = self._host_pool_structs(types, inst)
        count = C.c_int64(0)
        self._check(self._lib.gs_risk_scan_host(
            self._h, _host_ptr(assigned_inst, np.int32, n, "assigned_inst"),
            _host_ptr(generated_tokens, np.int32, n, "generated_tokens"),
            _host_ptr(pred_len, np.int32, n, "pred_len"),
            _host_ptr(elapsed_ms, np.float32, n, "elapsed_ms"), _host_ptr(slo_ms, np.float32, n, "slo_ms"), n,
            C.byref(hi), C.byref(ht), _host_ptr(out_flag_bits, np.uint32, (n + 31) // 32, "out_flag_bits"),
            _host_ptr(out_cand_idx, np.int32, cap, "out_cand_idx"), cap,
            C.cast(C.byref(count), C.c_void_p), self._stream(stream)))
        return int(count.value)

    def device_status(self, stream=None) -> int:
        bits = C.c_uint(0)
        self._check(self._lib.gs_device_status(self._h, self._stream(stream), C.byref(bits)))
        return int(bits.value)

    def eval_counters(self, clear: bool = True, stream=None):
        """Work counters of the routing kernels (all zero unless the library was built with
        -DGS_COUNT_EVALS): exact scorings, row bounds, type bounds, queued, fallback, exhaustive."""
        out = (C.c_uint64 * 8)()
        self._check(self._lib.gs_eval_counters(self._h, self._stream(stream), out, 1 if clear else 0))
        return [int(v) for v in out]

    def launch_count(self) -> int:
        return int(self._lib.gs_launch_count(self._h))

    def timing_enable(self, on: bool):
        self._check(self._lib.gs_timing_enable(self._h, 1 if on else 0))

    def timing_read(self, kernel: int):
        """(total milliseconds, launches) of one kernel since timing was enabled."""
        ms, n = C.c_double(0.0), C.c_int64(0)
        self._check(self._lib.gs_timing_read(self._h, int(kernel), C.byref(ms), C.byref(n)))
        return float(ms.value), int(n.value)

    def last_cuda_error(self) -> int:
        return int(self._lib.gs_last_cuda_error(self._h))


NOALLOC_MAX_ACTIVE = 16_777_216


def risk_scan_noalloc(assigned_inst, generated_tokens, pred_len, elapsed_ms, slo_ms, pool: InstancePool,
                      out_flag_bits, out_cand_idx, out_cand_count, out_status_bits=None,
                      cand_capacity: Optional[int] = None, n_active: Optional[int] = None, stream=None):
    """gs_risk_scan_noalloc: the risk scan for callers that must not allocate device memory.

    Needs no GoodServe context (creating one allocates).  The scan's scratch is a fixed array
    inside the library, shared by every call on the same GPU, so calls on one GPU must not
    overlap; at most NOALLOC_MAX_ACTIVE requests per call.  Runs on the tensors' device, which
    must be the current CUDA device.  This wrapper allocates nothing either: every tensor,
    including the optional one-word ``out_status_bits`` (int32, zeroed by the caller), is the
    caller's.
    """
    lib = load_library()
    n = int(assigned_inst.numel()) if n_active is None else int(n_active)
    cap = (0 if out_cand_idx is None else int(out_cand_idx.numel())) if cand_capacity is None else int(cand_capacity)
    dev = assigned_inst.device
    if torch.cuda.current_device() != dev.index:
        raise ValueError("risk_scan_noalloc runs on the current device; make the tensors' device current")
    i32, f32 = torch.int32, torch.float32
    M, Tn = pool.n_instances, pool.n_types
    inst = _Instances(_dev_ptr(pool.type_id, i32, M, "type_id", dev),
                      _dev_ptr(pool.queued_prefill_tokens, i32, M, "queued_prefill_tokens", dev),
                      _dev_ptr(pool.decode_batch, i32, M, "decode_batch", dev),
                      _dev_ptr(pool.free_kv_tokens, i32, M, "free_kv_tokens", dev),
                      _dev_ptr(pool.q_ema_ms, f32, M, "q_ema_ms", dev), M)
    types = _Types(_dev_ptr(pool.prefill_ms_per_tok, f32, Tn, "prefill_ms_per_tok", dev),
                   _dev_ptr(pool.tpot_a_ms, f32, Tn, "tpot_a_ms", dev),
                   _dev_ptr(pool.tpot_b_ms, f32, Tn, "tpot_b_ms", dev), Tn)
    s = torch.cuda.current_stream(dev) if stream is None else stream
    rc = lib.gs_risk_scan_noalloc(
        _dev_ptr(assigned_inst, i32, n, "assigned_inst", dev),
        _dev_ptr(generated_tokens, i32, n, "generated_tokens", dev),
        _dev_ptr(pred_len, i32, n, "pred_len", dev),
        _dev_ptr(elapsed_ms, f32, n, "elapsed_ms", dev),
        _dev_ptr(slo_ms, f32, n, "slo_ms", dev), n,
        C.byref(inst), C.byref(types),
        _dev_ptr(out_flag_bits, i32, (n + 31) // 32, "out_flag_bits", dev),
        _dev_ptr(out_cand_idx, i32, cap, "out_cand_idx", dev), cap,
        _dev_ptr(out_cand_count, torch.int64, 1, "out_cand_count", dev),
        _dev_ptr(out_status_bits, i32, 1, "out_status_bits", dev), s.cuda_stream or None)
    if rc != 0:
        raise GoodServeError(rc, lib.gs_strerror(rc).decode())
