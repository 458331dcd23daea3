"""ctypes binding of include/cleave.h.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
lib_path = os.path.join(_HERE, "lib", "libcleave.so")

if not os.path.exists(lib_path):
    raise ImportError(
        f"{lib_path} is missing: build it with `python -m paper_2512_22142_b200.build` "
        "(or __graft_entry__.build()); there is no fallback implementation")
lib = C.CDLL(lib_path)

# numpy mirrors of the C records
DEVICE_DTYPE = np.dtype([(n, "<u8") for n in
                         ("mem_bytes", "flops_mflops", "dl_Bps", "ul_Bps", "dl_lat_ns", "ul_lat_ns")])
GEMM_DTYPE = np.dtype([("M", "<u4"), ("N", "<u4"), ("K", "<u4"), ("lda", "<u4"), ("ldb", "<u4"),
                       ("transA", "u1"), ("transB", "u1"), ("level", "<u2")])
TASK_DTYPE = np.dtype([(n, "<u4") for n in
                       ("id", "gemm", "dev", "parent", "m0", "m1", "n0", "n1", "k0", "k1", "kslice", "flags")]
                      + [("part_off", "<u8"), ("cost_ns", "<u8")])
assert DEVICE_DTYPE.itemsize == 48 and GEMM_DTYPE.itemsize == 24 and TASK_DTYPE.itemsize == 64


class Opts(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("gran_m", "gran_n", "gran_k", "kslice_max", "ksplit",
                                          "ksplit_cap", "reissue_fanout", "b_in", "b_out", "tail_alpha_milli", "tail_beta_ppm")]


_vp, _u32, _u64, _i = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int
_sig = {
    "cleave_plan_opts_default": (None, [C.POINTER(Opts)]),
    "cleave_plan": (_i, [_vp, _u32, _vp, _u32, C.POINTER(Opts), C.POINTER(_vp)]),
    "cleave_plan_uniform": (_i, [_vp, _u32, _u32, _u32, _u32, C.POINTER(Opts), C.POINTER(_vp)]),
    "cleave_plan_num_tasks": (_u32, [_vp]),
    "cleave_plan_num_original": (_u32, [_vp]),
    "cleave_plan_tasks": (_vp, [_vp]),
    "cleave_plan_arena_elems": (_u64, [_vp]),
    "cleave_plan_ksplit": (_u32, [_vp, _u32]),
    "cleave_plan_makespan_ns": (_u64, [_vp, _u32]),
    "cleave_plan_tstar_ns": (_u64, [_vp, _u32]),
    "cleave_plan_num_tiles": (_u32, [_vp]),
    "cleave_plan_num_launches": (_u32, [_vp]),
    "cleave_plan_num_levels": (_u32, [_vp]),
    "cleave_plan_finishable": (_u32, [_vp, _u32]),
    "cleave_plan_level_makespan_ns": (_u64, [_vp, _u32]),
    "cleave_plan_step_makespan_ns": (_u64, [_vp]),
    "cleave_exec_opts": (_i, [_vp, _vp, _vp, _vp, _vp, _u32, _u32, _u32, _vp]),
    "cleave_set_wait_limit_ns": (_i, [_vp, _u64]),
    "cleave_set_drops": (_i, [_vp, _vp, _u32]),
    "cleave_exec": (_i, [_vp, _vp, _vp, _vp, _vp]),
    "cleave_exec_fused": (_i, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "cleave_assemble": (_i, [_vp, _vp, _vp, _vp]),
    "cleave_assemble_static": (_i, [_vp, _vp, _vp, _vp]),
    "cleave_reissue": (_i, [_vp, _vp, _u32, _vp, _vp, _vp, _vp]),
    "cleave_replan": (_i, [_vp, _vp, _u32, C.POINTER(_u32)]),
    "cleave_verify": (_i, [_vp, _vp, _vp, _vp, _u64, C.c_float, C.POINTER(_u32), _vp]),
    "cleave_verify_values": (_i, [_vp, _vp]),
    "cleave_status": (_i, [_vp, _vp]),
    "cleave_done_counts": (_i, [_vp, _vp, _vp]),
    "cleave_task_num_tiles": (_u32, [_vp, _u32]),
    "cleave_last_kernel_ms": (_i, [_vp, C.POINTER(C.c_float), C.POINTER(C.c_float)]),
    "cleave_destroy": (None, [_vp]),
    "cleave_strerror": (C.c_char_p, [_i]),
}
for _name, (_res, _args) in _sig.items():
    _f = getattr(lib, _name)
    _f.restype, _f.argtypes = _res, _args


EXEC_DIRECT, EXEC_FINISH, EXEC_BF16, EXEC_CONSUME = 1, 2, 4, 8


def strerror(code: int) -> str:
    return lib.cleave_strerror(code).decode()


class CleaveError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {strerror(code)} ({code})")
        self.code = code


def _check(code: int, where: str):
    if code != 0:
        raise CleaveError(code, where)


def default_opts(**kw) -> Opts:
    o = Opts()
    lib.cleave_plan_opts_default(C.byref(o))
    for k, v in kw.items():
        if not hasattr(o, k):
            raise TypeError(f"unknown planner option {k}")
        setattr(o, k, int(v))
    return o


def gemm_array(gemms: Sequence) -> np.ndarray:
    """Accepts objects with M, N, K, transA, transB, lda, ldb attributes (or a ready array)."""
    if isinstance(gemms, np.ndarray) and gemms.dtype == GEMM_DTYPE:
        return np.ascontiguousarray(gemms)
    a = np.zeros(len(gemms), dtype=GEMM_DTYPE)
    for i, g in enumerate(gemms):
        a[i] = (g.M, g.N, g.K, g.lda, g.ldb, g.transA, g.transB, getattr(g, "level", 0))
    return a


def _ptr_array(tensors) -> np.ndarray:
    return np.array([t if isinstance(t, int) else t.data_ptr() for t in tensors], dtype=np.uint64)


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


class Plan:
    """Owns a cleave_plan_t.  Methods carry the names of the C entry points."""

    def __init__(self, handle: int, n_gemms: int):
        self._h = C.c_void_p(handle)
        self.n_gemms = n_gemms

    def close(self):
        if self._h:
            lib.cleave_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- host queries
    @property
    def num_tasks(self) -> int:
        return lib.cleave_plan_num_tasks(self._h)

    @property
    def num_original(self) -> int:
        return lib.cleave_plan_num_original(self._h)

    @property
    def num_tiles(self) -> int:
        return lib.cleave_plan_num_tiles(self._h)

    @property
    def num_launches(self) -> int:
        return lib.cleave_plan_num_launches(self._h)

    @property
    def arena_elems(self) -> int:
        return lib.cleave_plan_arena_elems(self._h)

    def tasks(self) -> np.ndarray:
        """Copy of the task table (structured array, TASK_DTYPE)."""
        n = self.num_tasks
        buf = (C.c_char * (n * TASK_DTYPE.itemsize)).from_address(lib.cleave_plan_tasks(self._h))
        return np.frombuffer(buf, dtype=TASK_DTYPE, count=n).copy()

    def ksplit(self, gemm: int) -> int:
        return lib.cleave_plan_ksplit(self._h, gemm)

    def makespan_ns(self, gemm: int) -> int:
        return lib.cleave_plan_makespan_ns(self._h, gemm)

    def tstar_ns(self, gemm: int) -> int:
        return lib.cleave_plan_tstar_ns(self._h, gemm)

    def task_num_tiles(self, task: int) -> int:
        return lib.cleave_task_num_tiles(self._h, task)

    # ---- churn
    def set_drops(self, ids) -> None:
        a = np.ascontiguousarray(ids, dtype=np.uint32)
        _check(lib.cleave_set_drops(self._h, a.ctypes.data, len(a)), "cleave_set_drops")

    # ---- device calls.  A, B, C: sequences of torch tensors (or raw device addresses), one per GEMM.
    def exec(self, A, B, partials, stream=None) -> None:
        pa, pb = _ptr_array(A), _ptr_array(B)
        _check(lib.cleave_exec(self._h, pa.ctypes.data, pb.ctypes.data, partials.data_ptr(), _stream(stream)),
               "cleave_exec")

    def exec_fused(self, A, B, partials, Cs, stream=None) -> None:
        pa, pb, pc = _ptr_array(A), _ptr_array(B), _ptr_array(Cs)
        _check(lib.cleave_exec_fused(self._h, pa.ctypes.data, pb.ctypes.data, partials.data_ptr(), pc.ctypes.data,
                                     _stream(stream)), "cleave_exec_fused")

    def exec_opts(self, A, B, partials, Cs=None, direct=False, finish=False, bf16=False, consume=False, level_begin=0,
                  level_end=0xFFFFFFFF, stream=None) -> None:
        """cleave_exec_opts: flags CLEAVE_EXEC_DIRECT / FINISH / BF16 and a range of DAG levels."""
        pa, pb = _ptr_array(A), _ptr_array(B)
        pc = _ptr_array(Cs) if Cs is not None else None
        flags = (EXEC_DIRECT if direct else 0) | (EXEC_FINISH if finish else 0) | (EXEC_BF16 if bf16 else 0) | \
            (EXEC_CONSUME if consume else 0)
        _check(lib.cleave_exec_opts(self._h, pa.ctypes.data, pb.ctypes.data, partials.data_ptr(),
                                    pc.ctypes.data if pc is not None else None, flags, level_begin, level_end,
                                    _stream(stream)), "cleave_exec_opts")

    def set_wait_limit_ns(self, ns: int) -> None:
        _check(lib.cleave_set_wait_limit_ns(self._h, int(ns)), "cleave_set_wait_limit_ns")

    def finishable(self, gemm: int) -> bool:
        return bool(lib.cleave_plan_finishable(self._h, gemm))

    @property
    def num_levels(self) -> int:
        return lib.cleave_plan_num_levels(self._h)

    def level_makespan_ns(self, level: int) -> int:
        return lib.cleave_plan_level_makespan_ns(self._h, level)

    @property
    def step_makespan_ns(self) -> int:
        return lib.cleave_plan_step_makespan_ns(self._h)

    def assemble(self, partials, Cs, stream=None) -> None:
        pc = _ptr_array(Cs)
        _check(lib.cleave_assemble(self._h, partials.data_ptr(), pc.ctypes.data, _stream(stream)), "cleave_assemble")

    def assemble_static(self, partials, Cs, stream=None) -> None:
        """cleave_assemble_static: the assembly for callers that must not allocate device memory (its
        tables live in a fixed array inside the library; plans too large for it raise E_TOOBIG)."""
        pc = _ptr_array(Cs)
        _check(lib.cleave_assemble_static(self._h, partials if isinstance(partials, int) else partials.data_ptr(),
                                          pc.ctypes.data, _stream(stream)), "cleave_assemble_static")

    def reissue(self, failed, A, B, partials, stream=None) -> None:
        f = np.ascontiguousarray(failed if failed is not None else [], dtype=np.uint32)
        pa, pb = _ptr_array(A), _ptr_array(B)
        _check(lib.cleave_reissue(self._h, f.ctypes.data if len(f) else None, len(f), pa.ctypes.data, pb.ctypes.data,
                                  partials.data_ptr(), _stream(stream)), "cleave_reissue")

    def replan(self, failed) -> int:
        """Host-only half of reissue; returns the id of the first replacement task."""
        f = np.ascontiguousarray(failed, dtype=np.uint32)
        first = C.c_uint32(0)
        _check(lib.cleave_replan(self._h, f.ctypes.data if len(f) else None, len(f), C.byref(first)), "cleave_replan")
        return first.value

    def verify(self, A, B, partials, seed: int, tol: float = 2e-5, stream=None):
        """cleave_verify + cleave_verify_values: (number of flagged tasks, float32 array [n_tasks, 4] of
        lhs, rhs, scale, flag)."""
        pa, pb = _ptr_array(A), _ptr_array(B)
        bad = C.c_uint32(0)
        n = self.num_tasks
        _check(lib.cleave_verify(self._h, pa.ctypes.data, pb.ctypes.data, partials.data_ptr(), seed, tol, C.byref(bad),
                                 _stream(stream)), "cleave_verify")
        vals = np.zeros((n, 4), dtype=np.float32)
        _check(lib.cleave_verify_values(self._h, vals.ctypes.data), "cleave_verify_values")
        return bad.value, vals

    def status(self, stream=None) -> int:
        return lib.cleave_status(self._h, _stream(stream))

    def check_status(self, stream=None) -> None:
        _check(self.status(stream), "cleave_status")

    def done_counts(self, stream=None) -> np.ndarray:
        out = np.zeros(self.num_tasks, dtype=np.uint32)
        _check(lib.cleave_done_counts(self._h, out.ctypes.data, _stream(stream)), "cleave_done_counts")
        return out

    def last_kernel_ms(self):
        e, a = C.c_float(0), C.c_float(0)
        _check(lib.cleave_last_kernel_ms(self._h, C.byref(e), C.byref(a)), "cleave_last_kernel_ms")
        return e.value, a.value


def plan(gemms, devices: np.ndarray, opts: Optional[Opts] = None) -> Plan:
    """cleave_plan.  `devices`: uint64 array [n, 6] (mem, MFLOP/s, down B/s, up B/s, down ns, up ns)."""
    g = gemm_array(gemms)
    d = np.ascontiguousarray(devices, dtype=np.uint64).reshape(-1, 6)
    h = C.c_void_p()
    _check(lib.cleave_plan(g.ctypes.data, len(g), d.ctypes.data if len(d) else None, len(d),
                           C.byref(opts) if opts is not None else None, C.byref(h)), "cleave_plan")
    return Plan(h.value, len(g))


def plan_uniform(gemms, grid_m: int, grid_n: int, ksplit: int, opts: Optional[Opts] = None) -> Plan:
    g = gemm_array(gemms)
    h = C.c_void_p()
    _check(lib.cleave_plan_uniform(g.ctypes.data, len(g), grid_m, grid_n, ksplit,
                                   C.byref(opts) if opts is not None else None, C.byref(h)), "cleave_plan_uniform")
    return Plan(h.value, len(g))
