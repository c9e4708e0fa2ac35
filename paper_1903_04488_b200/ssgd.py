"""Thin ctypes binding over libssgd.so, the C-ABI CUDA library (include/ssgd.h).

Argument marshalling only: torch tensors supply device pointers and the current stream; every step
of the method runs inside the library's kernels.  There is no CPU fallback: if the library cannot be
loaded, importing a function from here raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libssgd.so")

OK, EINVAL, EALIGN, ENOTBOUND, EWORKSPACE, ECUDA, EDEVICE, ENOMEM, ETOOBIG, EPENDING = 0, -1, -2, -3, -4, -5, -6, -7, -8, -9
STATIC_MAX_NCAND = 262144
INSERT_AUTO, INSERT_GLOBAL, INSERT_SMEM, INSERT_TMA = 0, 1, 2, 3
PRUNE_AUTO, PRUNE_OFF, PRUNE_ON, PRUNE_EARLY_EXIT, PRUNE_FUSED = 0, 1, 2, 3, 4
STREAM_AUTO, STREAM_EVICT_FIRST, STREAM_L2_ONLY = 0, 1, 2
ZERO_DEFERRED, ZERO_EAGER = 0, 1
SCHED_AUTO, SCHED_COORDINATE_MAJOR, SCHED_WORKER_MAJOR = 0, 1, 2
FMT_F16, FMT_BF16 = 0, 1
MAX_R = 15

# name -> argument types, exactly the declarations of include/ssgd.h
_vp, _i64, _i32, _u64, _f32, _sz = C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_float, C.c_size_t
SIGNATURES = {
    "ssgd_create": [C.POINTER(_vp), _i64, _i32, _i64, _i64, _i32, _u64],
    "ssgd_destroy": [_vp],
    "ssgd_get_hash_params": [_vp, _vp],
    "ssgd_set_hash_params": [_vp, _vp],
    "ssgd_set_insert_mode": [_vp, _i32],
    "ssgd_set_prune_mode": [_vp, _i32],
    "ssgd_set_accumulate_schedule": [_vp, _i32],
    "ssgd_set_insert_split": [_vp, _i64],
    "ssgd_set_stream_loads": [_vp, _i32],
    "ssgd_set_prune_sample_rank": [_vp, _i64],
    "ssgd_set_table_persistence": [_vp, _i32],
    "ssgd_step_used_fallback": [_vp, _vp, C.POINTER(_i32)],
    "ssgd_set_zero_mode": [_vp, _i32],
    "ssgd_set_wait_limit_ns": [_vp, _i64],
    "ssgd_tail_trace": [_vp, _vp, C.POINTER(_i64)],
    "ssgd_test_withhold_block": [_vp, _i32],
    "ssgd_flush": [_vp, _vp],
    "ssgd_workspace_bytes": [_vp, _i64, C.POINTER(_sz)],
    "ssgd_bind": [_vp, _vp, _vp, _i64, _vp, _sz, _i64],
    "ssgd_unbind": [_vp],
    "ssgd_sketch_accumulate": [_vp, _vp, _i64, _f32, _vp, _vp],
    "ssgd_sketch_merge": [_vp, _vp, _vp, _vp],
    "ssgd_sketch_quantize16": [_vp, _vp, _i32, _vp, _vp],
    "ssgd_sketch_merge16": [_vp, _vp, _i32, _vp, _vp],
    "ssgd_unsketch_candidates": [_vp, _vp, _i64, _vp, _vp, _vp, _vp],
    "ssgd_exact_topk": [_vp, _vp, _i64, _vp, _vp, _vp],
    "ssgd_step": [_vp, _vp, _i64, _f32, _i64, _vp, _vp, _vp],
    "ssgd_step_host": [_vp, _vp, _i64, _f32, _i64, _vp, _vp, _vp, _vp],
    "ssgd_heavymix": [_vp, _vp, _u64, _vp, _vp, _vp, _vp, _vp],
    "ssgd_step_buffers": [_vp, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp)],
    "ssgd_hashes": [_vp, _vp, _i64, _vp, _vp, _vp],
    "ssgd_exact_topk_static": [_vp, _i64, _i32, _i64, _vp, _i64, _i64, _vp, _vp, _vp],
    "ssgd_set_timing": [_vp, _i32],
    "ssgd_get_stage_times": [_vp, _vp, C.POINTER(C.c_double), C.POINTER(_i64)],
    "ssgd_launch_count": [_vp, C.POINTER(_i64)],
    "ssgd_status": [_vp, _vp],
}

_lib = None


def lib() -> C.CDLL:
    """The loaded library.  Raises if it has not been built: there is nothing to fall back to."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_1903_04488_b200.build`")
        l = C.CDLL(LIB_PATH)
        for name, args in SIGNATURES.items():
            fn = getattr(l, name)
            fn.argtypes = args
            fn.restype = C.c_int
        l.ssgd_strerror.argtypes = [C.c_int]
        l.ssgd_strerror.restype = C.c_char_p
        l.ssgd_last_error.argtypes = [_vp]
        l.ssgd_last_error.restype = C.c_char_p
        _lib = l
    return _lib


class SsgdError(RuntimeError):
    def __init__(self, code: int, what: str, detail: str = ""):
        self.code = code
        msg = lib().ssgd_strerror(code).decode()
        super().__init__(f"{what}: {msg} ({code})" + (f": {detail}" if detail else ""))


def _dev_ptr(t: torch.Tensor | None, dtype, name: str):
    if t is None:
        return None
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: need a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def exact_topk_static(v: torch.Tensor, d: int, cand_idx: torch.Tensor, k: int, out_idx: torch.Tensor,
                      out_val: torch.Tensor) -> None:
    """Second round + final top-k on the library's built-in scratch: no workspace, no context, no allocation
    (for callers that may not allocate device memory; at most STATIC_MAX_NCAND candidates).  Does not zero
    any state.  Calls on one GPU must not overlap: they share that scratch."""
    code = lib().ssgd_exact_topk_static(_dev_ptr(v, torch.float32, "v"), v.shape[1], v.shape[0], d,
                                        _dev_ptr(cand_idx, torch.int32, "cand_idx"), cand_idx.numel(), k,
                                        _dev_ptr(out_idx, torch.int32, "out_idx"),
                                        _dev_ptr(out_val, torch.float32, "out_val"), _stream())
    if code:
        raise SsgdError(code, "ssgd_exact_topk_static")


class Ssgd:
    """One problem shape (d, r, c, k, W, seed); method names follow the C ABI."""

    def __init__(self, d: int, r: int, c: int, k: int, W: int, seed: int):
        self._lib = lib()
        h = _vp()
        code = self._lib.ssgd_create(C.byref(h), d, r, c, k, W, seed)
        if code:
            raise SsgdError(code, "ssgd_create")
        self._h = h
        self.d, self.r, self.c, self.k, self.W, self.seed = d, r, c, k, W, seed
        self._keep = None  # tensors bound to the context stay referenced here
        self.zero_mode = ZERO_DEFERRED

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and self._lib.ssgd_destroy(h) == EPENDING:
            # the object goes away with a deferred zero-out pending: the bound tensors are still referenced
            # here, so apply it to them; if that is no longer possible (interpreter shutdown), give it up
            try:
                code = self._lib.ssgd_flush(h, _stream())
            except Exception:
                code = ECUDA
            if code != OK:
                self._lib.ssgd_unbind(h)
            self._lib.ssgd_destroy(h)

    def _chk(self, code: int, what: str):
        if code:
            raise SsgdError(code, what, self._lib.ssgd_last_error(self._h).decode())

    # ---- host-only calls ---------------------------------------------------------------------
    def get_hash_params(self) -> torch.Tensor:
        out = (C.c_uint32 * (4 * self.r))()
        self._chk(self._lib.ssgd_get_hash_params(self._h, out), "ssgd_get_hash_params")
        return torch.tensor(list(out), dtype=torch.int64).reshape(self.r, 4)

    def set_hash_params(self, p) -> None:
        flat = [int(x) for row in p for x in row]
        arr = (C.c_uint32 * (4 * self.r))(*flat)
        self._chk(self._lib.ssgd_set_hash_params(self._h, arr), "ssgd_set_hash_params")

    def set_insert_mode(self, mode: int) -> None:
        self._chk(self._lib.ssgd_set_insert_mode(self._h, mode), "ssgd_set_insert_mode")

    def set_prune_mode(self, mode: int) -> None:
        self._chk(self._lib.ssgd_set_prune_mode(self._h, mode), "ssgd_set_prune_mode")

    def set_accumulate_schedule(self, mode: int) -> None:
        self._chk(self._lib.ssgd_set_accumulate_schedule(self._h, mode), "ssgd_set_accumulate_schedule")

    def set_prune_sample_rank(self, rank: int) -> None:
        self._chk(self._lib.ssgd_set_prune_sample_rank(self._h, rank), "ssgd_set_prune_sample_rank")

    def set_stream_loads(self, mode: int) -> None:
        self._chk(self._lib.ssgd_set_stream_loads(self._h, mode), "ssgd_set_stream_loads")

    def set_insert_split(self, nbytes: int) -> None:
        self._chk(self._lib.ssgd_set_insert_split(self._h, nbytes), "ssgd_set_insert_split")

    def set_table_persistence(self, enable: bool) -> None:
        self._chk(self._lib.ssgd_set_table_persistence(self._h, 1 if enable else 0), "ssgd_set_table_persistence")

    def set_wait_limit_ns(self, ns: int) -> None:
        self._chk(self._lib.ssgd_set_wait_limit_ns(self._h, ns), "ssgd_set_wait_limit_ns")

    def test_withhold_block(self, block_plus_one: int) -> None:
        self._chk(self._lib.ssgd_test_withhold_block(self._h, block_plus_one), "ssgd_test_withhold_block")

    def set_zero_mode(self, mode: int) -> None:
        self._chk(self._lib.ssgd_set_zero_mode(self._h, mode), "ssgd_set_zero_mode")
        self.zero_mode = mode

    def flush(self) -> None:
        """Applies a deferred zero-out (Algorithm 3 line 13) to the bound u and v on the current stream."""
        self._chk(self._lib.ssgd_flush(self._h, _stream()), "ssgd_flush")

    def step_used_fallback(self):
        """(redone without pruning?, survivors on the list, prune threshold bin) of the last step."""
        out = (_i32 * 5)()
        self._chk(self._lib.ssgd_step_used_fallback(self._h, _stream(), out), "ssgd_step_used_fallback")
        return bool(out[0]), int(out[1]), int(out[2])

    def step_first_pass(self):
        """(bucket bitmap too dense and the table was read instead?, set bits of the measured bitmap) of the last step."""
        out = (_i32 * 5)()
        self._chk(self._lib.ssgd_step_used_fallback(self._h, _stream(), out), "ssgd_step_used_fallback")
        return bool(out[3]), int(out[4])

    def tail_trace(self):
        """Nanosecond stamps of the last fused tail (see ssgd_tail_trace), -1 where none was taken."""
        out = (_i64 * 12)()
        self._chk(self._lib.ssgd_tail_trace(self._h, _stream(), out), "ssgd_tail_trace")
        return list(out)

    def workspace_bytes(self, ncand_max: int) -> int:
        out = _sz()
        self._chk(self._lib.ssgd_workspace_bytes(self._h, ncand_max, C.byref(out)), "ssgd_workspace_bytes")
        return out.value

    def set_timing(self, enable: bool) -> None:
        self._chk(self._lib.ssgd_set_timing(self._h, 1 if enable else 0), "ssgd_set_timing")

    def get_stage_times(self):
        """(ms per stage summed over the recorded steps [4], number of steps); waits for the stream."""
        ms = (C.c_double * 4)()
        n = _i64()
        self._chk(self._lib.ssgd_get_stage_times(self._h, _stream(), ms, C.byref(n)), "ssgd_get_stage_times")
        return list(ms), n.value

    def launch_count(self) -> int:
        out = _i64()
        self._chk(self._lib.ssgd_launch_count(self._h, C.byref(out)), "ssgd_launch_count")
        return out.value

    # ---- binding -----------------------------------------------------------------------------
    def bind(self, u: torch.Tensor, v: torch.Tensor, ncand_max: int, workspace: torch.Tensor | None = None):
        """Attach u, v ([W][ld] fp32 CUDA) and a workspace (uint8 CUDA; allocated here if None)."""
        if u.shape != v.shape or u.dim() != 2 or u.shape[0] != self.W:
            raise ValueError("u, v: need one shape [W][ld]")
        if workspace is None:
            workspace = torch.empty(self.workspace_bytes(ncand_max), dtype=torch.uint8, device=u.device)
        self._chk(self._lib.ssgd_bind(self._h, _dev_ptr(u, torch.float32, "u"), _dev_ptr(v, torch.float32, "v"),
                                      u.shape[1], _dev_ptr(workspace, torch.uint8, "workspace"),
                                      workspace.numel(), ncand_max), "ssgd_bind")
        self._keep = (u, v, workspace)
        self.ncand_max = ncand_max
        return workspace

    def unbind(self) -> None:
        """Detaches u, v and the workspace; a pending deferred zero-out is discarded."""
        self._chk(self._lib.ssgd_unbind(self._h), "ssgd_unbind")
        self._keep = None

    # ---- stage calls (asynchronous on the current stream) ------------------------------------
    def sketch_accumulate(self, g: torch.Tensor, rho: float, tables: torch.Tensor) -> None:
        self._chk(self._lib.ssgd_sketch_accumulate(self._h, _dev_ptr(g, torch.float32, "g"), g.shape[1], rho,
                                                   _dev_ptr(tables, torch.float32, "tables"), _stream()),
                  "ssgd_sketch_accumulate")

    def sketch_merge(self, tables: torch.Tensor, merged: torch.Tensor) -> None:
        self._chk(self._lib.ssgd_sketch_merge(self._h, _dev_ptr(tables, torch.float32, "tables"),
                                              _dev_ptr(merged, torch.float32, "merged"), _stream()),
                  "ssgd_sketch_merge")

    def sketch_quantize16(self, tables: torch.Tensor, fmt: int, q16: torch.Tensor) -> None:
        """tables [W][r][c] fp32 -> q16 [W][r][c] int16 (the 16-bit encodings), round to nearest even."""
        self._chk(self._lib.ssgd_sketch_quantize16(self._h, _dev_ptr(tables, torch.float32, "tables"), fmt,
                                                   _dev_ptr(q16, torch.int16, "q16"), _stream()), "ssgd_sketch_quantize16")

    def sketch_merge16(self, q16: torch.Tensor, fmt: int, merged: torch.Tensor) -> None:
        self._chk(self._lib.ssgd_sketch_merge16(self._h, _dev_ptr(q16, torch.int16, "q16"), fmt,
                                                _dev_ptr(merged, torch.float32, "merged"), _stream()), "ssgd_sketch_merge16")

    def unsketch_candidates(self, merged, ncand, cand_idx, cand_est=None, est_all=None) -> None:
        self._chk(self._lib.ssgd_unsketch_candidates(
            self._h, _dev_ptr(merged, torch.float32, "merged"), ncand, _dev_ptr(cand_idx, torch.int32, "cand_idx"),
            _dev_ptr(cand_est, torch.float32, "cand_est"), _dev_ptr(est_all, torch.float32, "est_all"), _stream()),
            "ssgd_unsketch_candidates")

    def exact_topk(self, cand_idx, out_idx, out_val) -> None:
        self._chk(self._lib.ssgd_exact_topk(self._h, _dev_ptr(cand_idx, torch.int32, "cand_idx"), cand_idx.numel(),
                                            _dev_ptr(out_idx, torch.int32, "out_idx"),
                                            _dev_ptr(out_val, torch.float32, "out_val"), _stream()),
                  "ssgd_exact_topk")

    def step(self, g: torch.Tensor, rho: float, ncand: int, out_idx: torch.Tensor, out_val: torch.Tensor) -> None:
        self._chk(self._lib.ssgd_step(self._h, _dev_ptr(g, torch.float32, "g"), g.shape[1], rho, ncand,
                                      _dev_ptr(out_idx, torch.int32, "out_idx"),
                                      _dev_ptr(out_val, torch.float32, "out_val"), _stream()), "ssgd_step")

    def heavymix(self, merged: torch.Tensor, fill_seed: int, out_idx: torch.Tensor, out_val: torch.Tensor,
                 l2_out: torch.Tensor | None = None, nheavy_out: torch.Tensor | None = None) -> None:
        """Algorithm 1 on a merged table: k coordinates (heavy ones + seeded random fill) and their exact sums."""
        self._chk(self._lib.ssgd_heavymix(self._h, _dev_ptr(merged, torch.float32, "merged"), fill_seed,
                                          _dev_ptr(out_idx, torch.int32, "out_idx"),
                                          _dev_ptr(out_val, torch.float32, "out_val"),
                                          _dev_ptr(l2_out, torch.float64, "l2_out"),
                                          _dev_ptr(nheavy_out, torch.int32, "nheavy_out"), _stream()), "ssgd_heavymix")

    def step_host(self, g_host: torch.Tensor, rho: float, ncand: int, g_stage: torch.Tensor,
                  out_idx_host: torch.Tensor, out_val_host: torch.Tensor) -> None:
        """g_host, out_*_host: CPU tensors (pinned for asynchronous copies); g_stage: CUDA staging buffer."""
        for t, dt, name in ((g_host, torch.float32, "g_host"), (out_idx_host, torch.int32, "out_idx_host"),
                            (out_val_host, torch.float32, "out_val_host")):
            if t.is_cuda or t.dtype != dt or not t.is_contiguous():
                raise TypeError(f"{name}: need a contiguous CPU tensor of {dt}")
        if g_host.shape != g_stage.shape:
            raise ValueError("g_host and g_stage must have one shape")
        self._chk(self._lib.ssgd_step_host(self._h, g_host.data_ptr(), g_host.shape[1], rho, ncand,
                                           _dev_ptr(g_stage, torch.float32, "g_stage"), out_idx_host.data_ptr(),
                                           out_val_host.data_ptr(), _stream()), "ssgd_step_host")

    def hashes(self, idx: torch.Tensor):
        n = idx.numel()
        h = torch.empty((self.r, n), dtype=torch.int32, device=idx.device)
        s = torch.empty((self.r, n), dtype=torch.int32, device=idx.device)
        self._chk(self._lib.ssgd_hashes(self._h, _dev_ptr(idx, torch.int32, "idx"), n, h.data_ptr(), s.data_ptr(),
                                        _stream()), "ssgd_hashes")
        return h, s

    def status(self) -> int:
        """Waits for the current stream; returns OK or EDEVICE (raises on a CUDA error)."""
        code = self._lib.ssgd_status(self._h, _stream())
        if code not in (OK, EDEVICE):
            self._chk(code, "ssgd_status")
        return code

    # ---- views of the workspace after ssgd_step (tests, diagnostics) --------------------------
    def step_buffers(self, ncand: int):
        """(merged [r][c], est [d], cand_idx [ncand], cand_xs [ncand]) as tensors aliasing the workspace."""
        ptrs = [_vp() for _ in range(4)]
        self._chk(self._lib.ssgd_step_buffers(self._h, *[C.byref(p) for p in ptrs]), "ssgd_step_buffers")
        ws = self._keep[2]
        base = ws.data_ptr()

        def view(p, n, dtype):
            off = p.value - base
            return ws[off: off + 4 * n].view(dtype)

        return (view(ptrs[0], self.r * self.c, torch.float32).view(self.r, self.c),
                view(ptrs[1], self.d, torch.float32), view(ptrs[2], ncand, torch.int32),
                view(ptrs[3], ncand, torch.float32))
