"""Seeded synthetic inputs for the ZGR step: parameter sets shaped like the paper's Transformer
workloads (RoBERTa, OPT and LLaMA families, Sec. 4 "Models"), subspaces, loss pairs, DTC payloads.

This module is the one piece shared by the CUDA path's tests/benchmark and the CPU oracle's
tests.  It holds none of the method's arithmetic: no counter-based generator, no Gaussian
transform, no mixing rule, no quantiser equation.  Random numbers come from numpy / torch library
generators; orthonormal bases come from a library QR.

No dataset, checkpoint or forward pass is involved anywhere: weights are N(0, 0.02^2) noise of
the right shapes and the loss pairs are seeded uniform numbers.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

DTYPE_CODES = {"f32": 0, "f16": 1, "bf16": 2}
DTYPE_BYTES = {"f32": 4, "f16": 2, "bf16": 2}


@dataclass(frozen=True)
class TensorSpec:
    name: str
    rows: int
    cols: int
    rank: int  # 0 for 1-D tensors (given as rows = 1)

    @property
    def numel(self) -> int:
        return self.rows * self.cols


@dataclass
class Workload:
    name: str
    dtype: str                   # "f32" | "f16" | "bf16"
    tensors: List[TensorSpec]
    rank: int
    alpha: float = 0.5           # Sec. 4 "FL Settings": alpha = 0.5 unless stated otherwise
    eps: float = 1e-3
    lr: float = 1e-4
    scale_mode: int = 1          # unit per-element variance (see the header of the C ABI)
    queries: int = 1             # perturbation queries per step, each with its own seed
    steps: int = 10
    dtc: bool = False            # guided coefficients delivered as int8 codes + per-row scales
    index: int = 0               # position in the list of configurations; seeds the loss stream
    fixed_losses: Optional[Tuple[float, float]] = None

    @property
    def params(self) -> int:
        return sum(t.numel for t in self.tensors)

    @property
    def coeffs(self) -> int:
        return sum(t.rank * t.cols for t in self.tensors)

    @property
    def bytes_per_sweep(self) -> int:
        """Algorithmic HBM traffic of one sweep: every weight read once and written once."""
        return 2 * DTYPE_BYTES[self.dtype] * self.params

    def seed(self, step: int, query: int) -> int:
        return 1000 * step + query

    def losses(self, step: int, query: int) -> Tuple[float, float]:
        """Loss pair (L+, L-) of one query: two independent U(1.5, 2.5) draws, seeded."""
        if self.fixed_losses is not None:
            return self.fixed_losses
        rng = np.random.default_rng([self.index, step, query])
        lp, lm = rng.uniform(1.5, 2.5, size=2)
        return float(lp), float(lm)


def _encoder_layer(prefix: str, d: int, ffn: int, r: int, norm_bias: bool = True) -> List[TensorSpec]:
    t = [TensorSpec(f"{prefix}.{n}.weight", d, d, r) for n in ("q", "k", "v", "o")]
    t += [TensorSpec(f"{prefix}.ffn_in.weight", ffn, d, r), TensorSpec(f"{prefix}.ffn_out.weight", d, ffn, r)]
    t += [TensorSpec(f"{prefix}.{n}.bias", 1, d, 0) for n in ("q", "k", "v", "o")]
    t += [TensorSpec(f"{prefix}.ffn_in.bias", 1, ffn, 0), TensorSpec(f"{prefix}.ffn_out.bias", 1, d, 0)]
    for n in ("ln1", "ln2"):
        t.append(TensorSpec(f"{prefix}.{n}.weight", 1, d, 0))
        if norm_bias:
            t.append(TensorSpec(f"{prefix}.{n}.bias", 1, d, 0))
    return t


def _llama_layer(prefix: str, d: int, ffn: int, r: int) -> List[TensorSpec]:
    t = [TensorSpec(f"{prefix}.{n}.weight", d, d, r) for n in ("q", "k", "v", "o")]
    t += [TensorSpec(f"{prefix}.gate.weight", ffn, d, r), TensorSpec(f"{prefix}.up.weight", ffn, d, r),
          TensorSpec(f"{prefix}.down.weight", d, ffn, r)]
    t += [TensorSpec(f"{prefix}.norm1.weight", 1, d, 0), TensorSpec(f"{prefix}.norm2.weight", 1, d, 0)]
    return t


def workload(name: str, layers: Optional[int] = None, vocab: Optional[int] = None) -> Workload:
    """The five configurations.  ``layers`` / ``vocab`` shrink a model for tests that replay every
    element on the CPU; shapes of the individual tensors are unchanged."""
    if name == "tiny":
        t = [TensorSpec(f"w{i}", 256, 256, 4) for i in range(4)] + [TensorSpec(f"b{i}", 1, 256, 0) for i in range(4)]
        return Workload("tiny", "f32", t, rank=4, steps=1, index=0, fixed_losses=(2.31, 2.29))
    if name == "roberta_large":
        L, V, r = layers or 24, vocab or 50265, 8
        t = [TensorSpec("embed.weight", V, 1024, r)]
        for i in range(L):
            t += _encoder_layer(f"l{i}", 1024, 4096, r)
        return Workload("roberta_large", "f32", t, rank=r, index=1)
    if name == "opt_1p3b":
        L, V, r = layers or 24, vocab or 50272, 16
        t = [TensorSpec("embed.weight", V, 2048, r)]
        for i in range(L):
            t += _encoder_layer(f"l{i}", 2048, 8192, r)
        t += [TensorSpec("final_ln.weight", 1, 2048, 0), TensorSpec("final_ln.bias", 1, 2048, 0)]
        return Workload("opt_1p3b", "f16", t, rank=r, index=2)
    if name == "llama_7b":
        L, V, r = layers or 32, vocab or 32000, 32
        t = [TensorSpec("embed.weight", V, 4096, r)]
        for i in range(L):
            t += _llama_layer(f"l{i}", 4096, 11008, r)
        t += [TensorSpec("final_norm.weight", 1, 4096, 0), TensorSpec("lm_head.weight", V, 4096, r)]
        return Workload("llama_7b", "bf16", t, rank=r, queries=4, index=3)
    if name == "llama_13b":
        L, V, r = layers or 40, vocab or 32000, 64
        t = [TensorSpec("embed.weight", V, 5120, r)]
        for i in range(L):
            t += _llama_layer(f"l{i}", 5120, 13824, r)
        t += [TensorSpec("final_norm.weight", 1, 5120, 0), TensorSpec("lm_head.weight", V, 5120, r)]
        return Workload("llama_13b", "bf16", t, rank=r, dtc=True, index=4)
    raise ValueError(f"unknown workload {name!r}")


WORKLOADS = ("tiny", "roberta_large", "opt_1p3b", "llama_7b", "llama_13b")


# ------------------------------------------------------------------------------------ host arrays
def subspace(rows: int, rank: int, seed: int) -> np.ndarray:
    """Orthonormal basis (rows x rank, fp32): QR of a seeded Gaussian in double, signs fixed so the
    diagonal of R is positive."""
    rng = np.random.default_rng([7, seed, rows, rank])
    q, r = np.linalg.qr(rng.standard_normal((rows, rank)))
    q = q * np.sign(np.diag(r))[None, :]
    return np.ascontiguousarray(q, dtype=np.float32)


def weights_host(spec: TensorSpec, seed: int) -> np.ndarray:
    """N(0, 0.02^2) weights as float64 (the caller rounds them to the storage type)."""
    rng = np.random.default_rng([11, seed, spec.rows, spec.cols])
    return 0.02 * rng.standard_normal((spec.rows, spec.cols))


def dtc_payload(rank: int, cols: int, seed: int):
    """Synthetic compressed coefficients: int8 codes with the spread of a unit Gaussian quantised
    over +-4.2 sigma, and per-row fp32 scales near 4.2/127.  Returns (codes, scales)."""
    rng = np.random.default_rng([13, seed, rank, cols])
    codes = np.clip(np.rint(rng.standard_normal((rank, cols)) * (127.0 / 4.2)), -127, 127).astype(np.int8)
    scales = ((4.2 / 127.0) * (1.0 + 0.1 * rng.uniform(-1.0, 1.0, size=rank))).astype(np.float32)
    return codes, scales


def sample_indices(numel: int, count: int, seed: int) -> np.ndarray:
    """Sorted unique linear indices into a tensor of ``numel`` elements."""
    rng = np.random.default_rng([17, seed, numel])
    if count >= numel:
        return np.arange(numel, dtype=np.int64)
    return np.unique(rng.integers(0, numel, size=count, dtype=np.int64))


# ------------------------------------------------------------------------------------ device tensors
def torch_dtype(name: str):
    import torch
    return {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[name]


@dataclass
class DeviceModel:
    """A workload materialised in device memory (torch tensors own the buffers)."""
    workload: Workload
    theta: list = field(default_factory=list)     # per tensor, (rows, cols) in the workload's dtype
    U: list = field(default_factory=list)         # per tensor, (rows, rank) fp32 or None
    q: list = field(default_factory=list)         # per tensor, (rank, cols) int8 or None
    scale: list = field(default_factory=list)     # per tensor, (rank,) fp32 or None


def materialise(wl: Workload, device, seed: int = 0) -> DeviceModel:
    """Weights drawn on the device with torch's generator; subspaces by QR on the host (they are
    small) and copied; DTC payloads on the host and copied."""
    import torch
    dm = DeviceModel(wl)
    gen = torch.Generator(device=device)
    td = torch_dtype(wl.dtype)
    for l, s in enumerate(wl.tensors):
        gen.manual_seed(1_000_003 * (seed + 1) + l)
        w = torch.empty((s.rows, s.cols), dtype=torch.float32, device=device)
        w.normal_(0.0, 0.02, generator=gen)
        dm.theta.append(w.to(td) if td != torch.float32 else w)
        del w
        if s.rank > 0:
            dm.U.append(torch.from_numpy(subspace(s.rows, s.rank, seed * 100_003 + l)).to(device))
            if wl.dtc:
                codes, scales = dtc_payload(s.rank, s.cols, seed * 100_003 + l)
                dm.q.append(torch.from_numpy(codes).to(device))
                dm.scale.append(torch.from_numpy(scales).to(device))
            else:
                dm.q.append(None)
                dm.scale.append(None)
        else:
            dm.U.append(None)
            dm.q.append(None)
            dm.scale.append(None)
    return dm
