"""Seeded synthetic inputs: transformer-layer GEMM lists, bf16 tensors, device records, failed ids.

This module serves both the CPU oracle and the CUDA library and therefore contains no arithmetic
of the method itself: it only names shapes, draws random tensors / device capabilities with fixed
seeds, and hands them out as plain arrays.  Everything random is produced here and passed to the
two sides as input.

Shapes follow the paper's transformer workloads (Table "Representative GEMMs ... in a single
transformer layer": projections tokens x d_in -> d_out; Section 2 "Device heterogeneity": 5-27
TFLOPS, 10-100 MB/s downlink, uplink 2-10x slower).  The paper's OPT / Llama-2 traces and its
device-capability data sets are not redistributed here; these synthetic stand-ins have the same
shapes and ranges.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

# Device record column order (all uint64): M_k, F_k, W^d_k, W^u_k, L^d_k, L^u_k
DEV_FIELDS = ("mem_bytes", "flops_mflops", "dl_Bps", "ul_Bps", "dl_lat_ns", "ul_lat_ns")

# Latency constants implied by the paper's worked example (Section 5.2, per-level cost of the
# 512-device Llama2-13B case): downlink overhead 5 ms, uplink overhead 10 ms.
DL_LAT_NS = 5_000_000
UL_LAT_NS = 10_000_000


@dataclass(frozen=True)
class GemmSpec:
    """One GEMM C[M x N] = op(A)[M x K] . op(B)[K x N] over row-major stored operands.

    transA = 0: A stored [M x K] (K contiguous);  transA = 1: A stored [K x M], A[i,k] = X[k,i].
    transB = 0: B stored [K x N] (N contiguous);  transB = 1: B stored [N x K], B[k,j] = W[j,k].
    lda / ldb are the row strides of the stored matrices, in elements.
    """
    name: str
    M: int
    N: int
    K: int
    transA: int
    transB: int
    lda: int
    ldb: int
    a_key: str
    b_key: str
    level: int = 0                         # DAG level: a GEMM may read what lower levels produced
    out_key: Optional[str] = None          # name under which the (bf16) result feeds higher levels

    @property
    def flops(self) -> int:
        return 2 * self.M * self.N * self.K


@dataclass(frozen=True)
class TensorSpec:
    rows: int
    cols: int
    std: float


@dataclass
class Workload:
    name: str
    gemms: List[GemmSpec]
    tensors: Dict[str, TensorSpec]
    n_devices: int = 0                     # 0: uniform plan (no device list)
    mem_range: Tuple[int, int] = (0, 0)     # bytes, log-uniform
    uniform: Optional[Tuple[int, int, int]] = None   # (grid_m, grid_n, ksplit)
    fail_frac: float = 0.0
    seed: int = 0
    note: str = ""
    produced: Dict[str, TensorSpec] = field(default_factory=dict)   # tensors written by GEMMs of the step

    @property
    def flops(self) -> int:
        return sum(g.flops for g in self.gemms)


def projection_gemms(tokens: int, projections: Sequence[Tuple[str, int, int]],
                     passes: Sequence[str] = ("fwd", "dgrad", "wgrad")):
    """GEMM list of one training step over linear layers `name: d_in -> d_out` on `tokens` rows.

    fwd   Y  = X . W        (M=tokens, N=d_out, K=d_in)   X[T x d_in], W[d_in x d_out]
    dgrad dX = dY . W^T     (M=tokens, N=d_in,  K=d_out)  B[k,j] = W[j,k]  -> transB = 1
    wgrad dW = X^T . dY     (M=d_in,   N=d_out, K=tokens) A[i,k] = X[k,i]  -> transA = 1
    """
    gemms: List[GemmSpec] = []
    tensors: Dict[str, TensorSpec] = {}
    for name, d_in, d_out in projections:
        tensors[f"{name}.X"] = TensorSpec(tokens, d_in, 1.0)
        tensors[f"{name}.W"] = TensorSpec(d_in, d_out, 0.02)
        tensors[f"{name}.dY"] = TensorSpec(tokens, d_out, 1.0)
    for p in passes:
        for name, d_in, d_out in projections:
            if p == "fwd":
                gemms.append(GemmSpec(f"{name}.fwd", tokens, d_out, d_in, 0, 0, d_in, d_out,
                                      f"{name}.X", f"{name}.W"))
            elif p == "dgrad":
                gemms.append(GemmSpec(f"{name}.dgrad", tokens, d_in, d_out, 0, 1, d_out, d_out,
                                      f"{name}.dY", f"{name}.W"))
            elif p == "wgrad":
                gemms.append(GemmSpec(f"{name}.wgrad", d_in, d_out, tokens, 1, 0, d_in, d_out,
                                      f"{name}.X", f"{name}.dY"))
            else:
                raise ValueError(p)
    return gemms, tensors


def attention_gemms(n_heads: int, seq: int, d_head: int):
    """The two GEMMs of every attention head (batch x heads of them are independent; the paper's
    table of representative GEMMs lists Q.K^T as 1024 x 128 x 1024, count 128 x 32):
      scores  S = Q . K^T   (M = seq, N = seq, K = d_head)   K stored [seq x d_head] -> transB = 1
      context O = P . V     (M = seq, N = d_head, K = seq)   P stands in for softmax(S) in bf16"""
    gemms: List[GemmSpec] = []
    tensors: Dict[str, TensorSpec] = {}
    for h in range(n_heads):
        tensors[f"h{h}.Q"] = TensorSpec(seq, d_head, 1.0)
        tensors[f"h{h}.K"] = TensorSpec(seq, d_head, 1.0)
        tensors[f"h{h}.P"] = TensorSpec(seq, seq, 0.05)
        tensors[f"h{h}.V"] = TensorSpec(seq, d_head, 1.0)
    for h in range(n_heads):
        gemms.append(GemmSpec(f"h{h}.qk", seq, seq, d_head, 0, 1, d_head, d_head, f"h{h}.Q", f"h{h}.K"))
    for h in range(n_heads):
        gemms.append(GemmSpec(f"h{h}.pv", seq, d_head, seq, 0, 0, seq, d_head, f"h{h}.P", f"h{h}.V"))
    return gemms, tensors


def two_branch_chain(tokens: int, d0: int, d1: int, d2: int):
    """A three-level DAG in the shape of a transformer block's dependencies (Section 4.1: GEMMs of a
    level are independent, the outputs of a level are the inputs of the next):
      level 0   Ha = X . Wa,  Hb = X . Wb          (two GEMMs sharing X, like the QKV projections)
      level 1   Ya = Ha . Va, Yb = Hb . Vb          (each reads one level-0 output as its A operand)
      level 2   G  = Ha^T . Hb                      (reads two level-0 outputs; contraction over tokens)
    Produced tensors are bf16, as a training step would keep its activations."""
    tensors = {"X": TensorSpec(tokens, d0, 1.0), "Wa": TensorSpec(d0, d1, 0.05), "Wb": TensorSpec(d0, d1, 0.05),
               "Va": TensorSpec(d1, d2, 0.05), "Vb": TensorSpec(d1, d2, 0.05)}
    produced = {"Ha": TensorSpec(tokens, d1, 0.0), "Hb": TensorSpec(tokens, d1, 0.0)}
    gemms = [
        GemmSpec("Ha", tokens, d1, d0, 0, 0, d0, d1, "X", "Wa", 0, "Ha"),
        GemmSpec("Hb", tokens, d1, d0, 0, 0, d0, d1, "X", "Wb", 0, "Hb"),
        GemmSpec("Ya", tokens, d2, d1, 0, 0, d1, d2, "Ha", "Va", 1, None),
        GemmSpec("Yb", tokens, d2, d1, 0, 0, d1, d2, "Hb", "Vb", 1, None),
        GemmSpec("G", d1, d1, tokens, 1, 0, d1, d1, "Ha", "Hb", 2, None),
    ]
    return gemms, tensors, produced


MB = 1 << 20
GB = 1 << 30


def gpt2_small_projections(d=768, ffn=3072):
    return [("qkv", d, 3 * d), ("out", d, d), ("fc1", d, ffn), ("fc2", ffn, d)]


def llama_projections(d, ffn):
    return [("q", d, d), ("k", d, d), ("v", d, d), ("o", d, d),
            ("gate", d, ffn), ("up", d, ffn), ("down", ffn, d)]


def config(i: int, scale: int = 1) -> Workload:
    """The five benchmark configurations.  `scale` > 1 divides the token count and the hidden
    sizes by `scale` (kept multiples of 8) to give a structurally identical small case that a
    CPU can finish in seconds."""
    def s(x, q=8):
        return max(q, (x // scale) // q * q)

    if i == 1:
        gemms, tensors = projection_gemms(256, [("lin", 768, 768)], passes=("fwd",))
        return Workload("cfg1-tiny-fwd", gemms, tensors, uniform=(4, 4, 2), seed=0,
                        note="single forward GEMM, uniform 4x4 blocks x 2 K-slices")
    if i == 2:
        gemms, tensors = projection_gemms(s(8192), gpt2_small_projections(s(768), s(3072)))
        return Workload("cfg2-gpt2-small-layer", gemms, tensors, n_devices=max(4, 64 // scale),
                        mem_range=(256 * MB, 4 * GB), seed=0)
    if i in (3, 4):
        gemms, tensors = projection_gemms(s(8192), llama_projections(s(4096), s(11008)))
        return Workload("cfg3-llama7b-layer" if i == 3 else "cfg4-llama7b-layer-churn",
                        gemms, tensors, n_devices=max(8, 1024 // (scale * scale)),
                        mem_range=(512 * MB, 8 * GB), fail_frac=0.10 if i == 4 else 0.0, seed=0)
    if i == 5:
        gemms, tensors = projection_gemms(s(16384), llama_projections(s(5120), s(13824)))
        return Workload("cfg5-llama13b-layer", gemms, tensors,
                        n_devices=max(8, 4096 // (scale * scale)),
                        mem_range=(128 * MB, 2 * GB), seed=0)
    if i == 6:
        # not one of the five benchmark configurations: the attention GEMMs of the paper's GEMM-shape
        # table (1024 x 128 x 1024 per head), many tiny independent GEMMs; 1024 heads at scale 1
        gemms, tensors = attention_gemms(max(2, 1024 // (scale * scale)), s(1024, 64), s(128, 64))
        return Workload("attention-gemms", gemms, tensors, n_devices=max(4, 64 // scale),
                        mem_range=(256 * MB, 4 * GB), seed=0)
    raise ValueError(f"no config {i}")


# ----------------------------------------------------------------------------------------------
# tensors
# ----------------------------------------------------------------------------------------------

def make_tensors(w: Workload, seed: Optional[int] = None, integer: bool = False, pin: bool = False):
    """bf16 CPU tensors for every operand of the workload, in dictionary (= GEMM list) order.

    Gaussian mode: fp32 `randn * std`, rounded to bf16 (round-to-nearest-even).
    Integer mode: values uniform in {-4..4} (exactly representable; every product and partial sum
    of a GEMM with K < 2^20 is then exact in fp32 as well as fp64).
    """
    import torch
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed if seed is None else seed)
    out = {}
    for key, ts in w.tensors.items():
        if integer:
            t = torch.randint(-4, 5, (ts.rows, ts.cols), generator=g, dtype=torch.int32).to(torch.bfloat16)
        else:
            t = (torch.randn(ts.rows, ts.cols, generator=g, dtype=torch.float32) * ts.std).to(torch.bfloat16)
        if pin:
            t = t.pin_memory()
        out[key] = t
    return out


def bf16_bits(t) -> np.ndarray:
    """The raw bf16 bit patterns of a torch bf16 CPU tensor as a uint16 NumPy array (no copy)."""
    import torch
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.view(torch.int16).numpy().view(np.uint16)


# ----------------------------------------------------------------------------------------------
# devices and failures
# ----------------------------------------------------------------------------------------------

def make_devices(n: int, mem_lo: int, mem_hi: int, seed: int) -> np.ndarray:
    """n device records, uint64 [n, 6] in DEV_FIELDS order, every value already an integer.

    mem log-uniform in [mem_lo, mem_hi]; F log-uniform in 5-27 TFLOPS (stored in MFLOP/s);
    downlink log-uniform in 10-100 MB/s; uplink = downlink / ratio, ratio uniform in [2, 10];
    latencies fixed at 5 ms down / 10 ms up.
    """
    rng = np.random.default_rng(seed)
    mem = np.exp(rng.uniform(np.log(mem_lo), np.log(mem_hi), n))
    flops = np.exp(rng.uniform(np.log(5e6), np.log(27e6), n))          # MFLOP/s
    dl = np.exp(rng.uniform(np.log(10e6), np.log(100e6), n))           # B/s
    ratio = rng.uniform(2.0, 10.0, n)
    ul = dl / ratio
    d = np.empty((n, 6), dtype=np.uint64)
    d[:, 0] = np.floor(mem).astype(np.uint64)
    d[:, 1] = np.floor(flops).astype(np.uint64)
    d[:, 2] = np.floor(dl).astype(np.uint64)
    d[:, 3] = np.maximum(1, np.floor(ul)).astype(np.uint64)
    d[:, 4] = DL_LAT_NS
    d[:, 5] = UL_LAT_NS
    return d


def workload_devices(w: Workload) -> Optional[np.ndarray]:
    if w.n_devices == 0:
        return None
    return make_devices(w.n_devices, w.mem_range[0], w.mem_range[1], w.seed + 1)


def homogeneous_devices(n: int, mem=8 * GB, flops=6_000_000, dl=55_000_000, ul=7_500_000) -> np.ndarray:
    """n identical devices with the paper's median edge-device parameters (Table of absolute
    per-batch times: 6 TFLOPS, 55 MB/s down, 7.5 MB/s up)."""
    d = np.empty((n, 6), dtype=np.uint64)
    d[:] = (mem, flops, dl, ul, DL_LAT_NS, UL_LAT_NS)
    return d


def make_failed_ids(n_tasks: int, frac: float, seed: int) -> np.ndarray:
    """Sorted uint32 task ids of a uniformly random `frac` of the tasks, without replacement."""
    k = int(round(frac * n_tasks))
    rng = np.random.default_rng(seed)
    ids = rng.choice(n_tasks, size=k, replace=False)
    return np.sort(ids).astype(np.uint32)
