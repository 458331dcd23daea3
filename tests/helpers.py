"""Shared test plumbing: the same seeded inputs go to the oracle (NumPy, fp64) and to the library
(torch tensors on the GPU).  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np

import cleave_inputs as ci
from oracle import numerics as nm
from oracle.cost import devices_from_array
from oracle.plan import Gemm, Opts, plan as oracle_plan, plan_uniform as oracle_plan_uniform

TASK_FIELDS = ("id", "gemm", "dev", "parent", "m0", "m1", "n0", "n1", "k0", "k1", "kslice", "flags",
               "part_off", "cost_ns")


def oracle_gemms(w):
    return [Gemm(g.M, g.N, g.K, g.transA, g.transB, getattr(g, "level", 0)) for g in w.gemms]


def oracle_plan_for(w, **opts):
    devs = ci.workload_devices(w)
    if devs is None:
        return oracle_plan_uniform(oracle_gemms(w), *w.uniform, Opts(**opts))
    return oracle_plan(oracle_gemms(w), devices_from_array(devs), Opts(**opts))


def lib_plan_for(w, **opts):
    import paper_2512_22142_b200 as cl
    devs = ci.workload_devices(w)
    if devs is None:
        return cl.plan_uniform(w.gemms, *w.uniform, cl.default_opts(**opts))
    return cl.plan(w.gemms, devs, cl.default_opts(**opts))


def task_matrix_lib(p) -> np.ndarray:
    t = p.tasks()
    return np.stack([t[n].astype(np.uint64) for n in TASK_FIELDS], axis=1)


def task_matrix_oracle(op) -> np.ndarray:
    return np.array([t.astuple() for t in op.tasks], dtype=np.uint64).reshape(-1, len(TASK_FIELDS))


def oracle_operands(w, tensors):
    """op(A) [M x K] and op(B) [K x N] of every GEMM as fp64 arrays (views where possible)."""
    wide = {k: nm.bf16_bits_to_f64(ci.bf16_bits(t)) for k, t in tensors.items()}
    A = [nm.op_a(wide[g.a_key], g.transA) for g in w.gemms]
    B = [nm.op_b(wide[g.b_key], g.transB) for g in w.gemms]
    return A, B


class GpuRun:
    """Device copies of the operands plus arena and outputs for one workload and plan."""

    def __init__(self, w, tensors, plan, poison=True, bf16_out=False):
        import torch
        self.torch = torch
        self.w, self.plan = w, plan
        dev = torch.device("cuda:0")
        self.dev_tensors = {k: t.to(dev) for k, t in tensors.items()}
        c_dtype = torch.bfloat16 if bf16_out else torch.float32
        # tensors the step itself produces (outputs of lower DAG levels that feed higher ones): bf16, NaN until written
        for k, spec in w.produced.items():
            self.dev_tensors[k] = torch.full((spec.rows, spec.cols), float("nan"), dtype=torch.bfloat16, device=dev)
        self.A = [self.dev_tensors[g.a_key] for g in w.gemms]
        self.B = [self.dev_tensors[g.b_key] for g in w.gemms]
        self.partials = torch.empty(max(1, plan.arena_elems), dtype=torch.float32, device=dev)
        if poison:
            self.partials.fill_(float("nan"))
        self.C = [self.dev_tensors[g.out_key] if g.out_key else
                  torch.full((g.M, g.N), float("nan"), dtype=c_dtype, device=dev) for g in w.gemms]

    def exec(self):
        self.plan.exec(self.A, self.B, self.partials)

    def exec_fused(self):
        self.plan.exec_fused(self.A, self.B, self.partials, self.C)

    def exec_opts(self, **kw):
        self.plan.exec_opts(self.A, self.B, self.partials, self.C, **kw)

    def assemble(self):
        self.plan.assemble(self.partials, self.C)

    def reissue(self, failed):
        self.plan.reissue(failed, self.A, self.B, self.partials)

    def results(self):
        """fp32 outputs as NumPy arrays; bf16 outputs as their uint16 bit patterns."""
        self.torch.cuda.synchronize()
        return [c.cpu().numpy() if c.dtype == self.torch.float32 else
                c.cpu().view(self.torch.int16).numpy().view(np.uint16) for c in self.C]


def assert_within_tolerance(C_gpu, C_ref, bound, rel_fro=1e-3, elem=1e-2, what=""):
    """Acceptance of the floating-point path: relative Frobenius error <= 1e-3 and
    |delta_ij| <= 1e-2 * (|A||B|)_ij."""
    d = C_gpu.astype(np.float64) - C_ref
    assert np.isfinite(C_gpu).all(), f"{what}: non-finite output"
    fro = np.linalg.norm(d) / max(np.linalg.norm(C_ref), 1e-300)
    assert fro <= rel_fro, f"{what}: relative Frobenius error {fro:.3e}"
    ratio = np.abs(d) / np.maximum(bound, 1e-300)
    assert ratio.max() <= elem, f"{what}: elementwise ratio {ratio.max():.3e}"
    return fro, ratio.max()
