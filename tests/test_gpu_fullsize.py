"""Full-size parity in the launch configuration the benchmark times (Llama-7B-shaped layer,
1024 devices): outputs the oracle can compute one by one, plus a Freivalds identity over the whole
of every C."""
import numpy as np
import pytest

import cleave_inputs as ci
from helpers import GpuRun, lib_plan_for
from oracle import check, numerics as nm

pytestmark = pytest.mark.gpu


def test_config3_sampled_entries_and_freivalds():
    import torch
    w = ci.config(3)
    ts = ci.make_tensors(w)
    p = lib_plan_for(w)
    run = GpuRun(w, ts, p)
    run.exec(); run.assemble(); p.check_status()
    torch.cuda.synchronize()
    rng = np.random.default_rng(7)
    wide = {}
    for gi, g in enumerate(w.gemms):
        for key in (g.a_key, g.b_key):
            if key not in wide:
                wide[key] = nm.bf16_bits_to_f64(ci.bf16_bits(ts[key]))
        A, B = nm.op_a(wide[g.a_key], g.transA), nm.op_b(wide[g.b_key], g.transB)
        C = run.C[gi].cpu().numpy()
        # 512 sampled entries, among them the four corners and tile-edge neighbours
        rows = np.concatenate([rng.integers(0, g.M, 500), [0, 0, g.M - 1, g.M - 1, 127, 128, 255, 256, 127, 128, 129, 63]])
        cols = np.concatenate([rng.integers(0, g.N, 500), [0, g.N - 1, 0, g.N - 1, 255, 256, 127, 128, 128, 127, 1, 64]])
        ref, bound = nm.sample_entries(A, B, rows, cols)
        got = C[rows, cols].astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-2 * bound), g.name
        assert np.linalg.norm(got - ref) <= 1e-3 * np.linalg.norm(ref), g.name
        worst, scale = check.freivalds_residual(A, B, C, seed=gi, reps=2)
        assert worst <= 1e-3 * scale, g.name     # any lost or doubled block shifts r^T C s far beyond rounding
