"""Seeded synthetic q/k/v streams shaped like long-response decoding.

This module only *draws inputs*.  It contains none of MorphKV's arithmetic (no
softmax, no scoring, no selection) so that both the CPU oracle's tests and the
CUDA path's tests can feed the very same materialised tensors to either side.

Every value is a pure function of ``(seed, tensor, layer, batch row, head,
position, element)``: a SplitMix64 stream (Steele, Lea & Flood 2014) is seeded
per row and turned into normals with Box-Muller.  Because nothing is
sequential, any (unit, position) can be regenerated at will, on any torch
device.  Parity runs materialise a tensor once and hand copies of it to both
sides, so ulp-level libm differences between devices cannot matter.

Value model
-----------
* ``v[., pos, :] ~ N(0, 1)``.
* ``k[., pos, :] = s * z`` with ``z ~ N(0,1)^d`` and ``s = 4`` with probability
  0.02 per row, else 1.  With ``sink=True`` the key at position 0 is scaled by
  a further factor 8 (an attention sink).
* ``q[hq, pos, :] = 0.5 * k[kv(hq), j, :] + z'`` where ``j`` is uniform over all
  earlier positions ``0..pos-1`` (whether or not still cached); ``q = z'`` at
  position 0.  This gives peaked, heavy-tailed attention.
* In bf16 mode every tensor is rounded to bf16 (round-to-nearest-even) once.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

_MASK64 = (1 << 64) - 1


def _s64(c: int) -> int:
    """Two's-complement view of an unsigned 64-bit constant as a Python int."""
    c &= _MASK64
    return c - (1 << 64) if c >= (1 << 63) else c


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)

# tensor tags
_TAG_K, _TAG_V, _TAG_QNOISE, _TAG_QPICK, _TAG_KHEAVY = 1, 2, 3, 4, 5


def _lsr(x: torch.Tensor, n: int) -> torch.Tensor:
    """Logical shift right on int64 tensors."""
    return (x >> n) & ((1 << (64 - n)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """SplitMix64 output function; int64 arithmetic wraps modulo 2**64."""
    x = (x ^ _lsr(x, 30)) * _M1
    x = (x ^ _lsr(x, 27)) * _M2
    return x ^ _lsr(x, 31)


def _uniform(bits: torch.Tensor) -> torch.Tensor:
    """53 random bits -> float64 in the open interval (0, 1)."""
    return (_lsr(bits, 11).to(torch.float64) + 0.5) * (2.0 ** -53)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One decode workload: shapes, MorphKV hyper-parameters and the seed."""

    name: str
    layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str  # "bf16" | "f32"
    prompt_len: int
    steps: int
    C: int
    R: int
    fusion: str  # "sum" | "max"
    seed: int
    sink: bool = False

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def units(self) -> int:
        return self.layers * self.batch * self.n_kv_heads

    @property
    def capacity(self) -> int:
        return self.C + self.R

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


_SEED0 = 0x25030979

WORKLOADS = {
    # tiny fp32 correctness case the CPU oracle finishes in seconds
    "c0": Workload("c0", 1, 1, 8, 2, 64, "f32", 256, 512, 64, 16, "sum", _SEED0 + 0),
    # Llama-3.1-8B-shaped attention stack, batch 1
    "c1": Workload("c1", 32, 1, 32, 8, 128, "bf16", 4096, 8192, 2000, 32, "max", _SEED0 + 1),
    # Mistral-7B-shaped, batch 32, attention-sink key at position 0
    "c2": Workload("c2", 32, 32, 32, 8, 128, "bf16", 2048, 4096, 1024, 32, "sum", _SEED0 + 2, sink=True),
    # long-response stress
    "c3": Workload("c3", 32, 8, 32, 8, 128, "bf16", 512, 32768, 4000, 64, "max", _SEED0 + 3),
}
for _C in (512, 1024, 2048, 4096, 8192):
    for _f in ("sum", "max"):
        WORKLOADS[f"c4_C{_C}_{_f}"] = Workload(
            f"c4_C{_C}_{_f}", 1, 128, 32, 8, 128, "bf16", _C + 32, 1024, _C, 32, _f, _SEED0 + 4)


# long prompts compressed into a 2K cache by one application of the policy (window 32, sum fusion): the setting of
# the paper's long-context runs, on the Llama-3.1-8B-shaped stack; `steps` decode steps follow in the parity tests
for _P in (6144, 32768, 131072):
    WORKLOADS[f"prefill_P{_P}"] = Workload(f"prefill_P{_P}", 32, 1, 32, 8, 128, "bf16", _P, 8, 2016, 32, "sum", _SEED0 + 5)

# the long-response setting with a window of 200 recent tokens inside a 4K budget, on the Llama-3.1-8B-shaped stack:
# 800 ring rows per unit, more than one tensor-core operand holds
WORKLOADS["w200"] = Workload("w200", 32, 1, 32, 8, 128, "bf16", 4096, 4096, 3896, 200, "sum", _SEED0 + 6)
# its prompt phase: a 6144-token prompt compressed into that budget (the 800 window rows are scored in four pieces)
WORKLOADS["prefill_w200_P6144"] = Workload("prefill_w200_P6144", 32, 1, 32, 8, 128, "bf16", 6144, 8, 3896, 200, "sum", _SEED0 + 7)


class Stream:
    """Counter-based generator of a workload's q/k/v at arbitrary positions.

    ``unit_slice`` style arguments (``layers``, ``batch``, ``heads``) are index
    tensors or ``None`` (all), so a test can draw the inputs of a few sampled
    units without materialising the rest.
    """

    def __init__(self, w: Workload, device: str | torch.device = "cpu"):
        self.w = w
        self.device = torch.device(device)

    # -- hashing ----------------------------------------------------------
    def _row_hash(self, tag: int, layer, batch, head, pos) -> torch.Tensor:
        """Hash of a row id; the arguments broadcast against each other."""
        h = torch.full((), _s64(self.w.seed * 0x100 + tag), dtype=torch.int64, device=self.device)
        h = _mix64(h + _GOLDEN)
        for field in (layer, batch, head, pos):
            h = _mix64((h ^ field) + _GOLDEN)
        return h

    def _normals(self, row_hash: torch.Tensor, d: int) -> torch.Tensor:
        """``d`` standard normals per row: Box-Muller on a SplitMix64 stream."""
        e = torch.arange(d, dtype=torch.int64, device=self.device)
        s = row_hash.unsqueeze(-1)
        u1 = _uniform(_mix64(s + _GOLDEN * (2 * e + 1)))
        u2 = _uniform(_mix64(s + _GOLDEN * (2 * e + 2)))
        return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)

    def _idx(self, n: int, sel: Optional[torch.Tensor]) -> torch.Tensor:
        if sel is None:
            return torch.arange(n, dtype=torch.int64, device=self.device)
        return torch.as_tensor(sel, dtype=torch.int64, device=self.device).reshape(-1)

    # -- raw (unrounded, float64) draws -------------------------------------
    def _k_raw(self, layer, batch, head, pos) -> torch.Tensor:
        """Keys for broadcastable index tensors -> [..., d] float64."""
        w = self.w
        z = self._normals(self._row_hash(_TAG_K, layer, batch, head, pos), w.head_dim)
        heavy = _uniform(self._row_hash(_TAG_KHEAVY, layer, batch, head, pos)) < 0.02
        scale = torch.where(heavy, 4.0, 1.0).to(torch.float64)
        if w.sink:
            scale = torch.where(pos == 0, scale * 8.0, scale)
        return z * scale.unsqueeze(-1)

    def _round(self, x: torch.Tensor) -> torch.Tensor:
        x = x.to(torch.float32)
        if self.w.dtype == "bf16":
            x = x.to(torch.bfloat16).to(torch.float32)
        return x

    # -- public draws -------------------------------------------------------
    def kv(self, positions, layers=None, batch=None, heads=None):
        """Keys and values at ``positions`` -> two float32 tensors [L,B,Hkv,len,d].

        The float32 values are exactly representable in the workload's dtype.
        """
        w = self.w
        li = self._idx(w.layers, layers)[:, None, None, None]
        bi = self._idx(w.batch, batch)[None, :, None, None]
        hi = self._idx(w.n_kv_heads, heads)[None, None, :, None]
        pi = torch.as_tensor(positions, dtype=torch.int64, device=self.device).reshape(-1)[None, None, None, :]
        li, bi, hi, pi = torch.broadcast_tensors(li, bi, hi, pi)
        k = self._k_raw(li, bi, hi, pi)
        v = self._normals(self._row_hash(_TAG_V, li, bi, hi, pi), w.head_dim)
        return self._round(k), self._round(v)

    def q(self, positions, layers=None, batch=None, kv_heads=None):
        """Queries at ``positions`` -> float32 [L,B,Hq_sel,len,d].

        ``kv_heads`` selects KV heads; the returned query heads are the GQA
        groups of those KV heads, in order (``G`` consecutive heads each).
        """
        w = self.w
        g = w.group
        kvh = self._idx(w.n_kv_heads, kv_heads)
        qh = (kvh[:, None] * g + torch.arange(g, dtype=torch.int64, device=self.device)[None, :]).reshape(-1)
        li = self._idx(w.layers, layers)[:, None, None, None]
        bi = self._idx(w.batch, batch)[None, :, None, None]
        hi = qh[None, None, :, None]
        pi = torch.as_tensor(positions, dtype=torch.int64, device=self.device).reshape(-1)[None, None, None, :]
        li, bi, hi, pi = torch.broadcast_tensors(li, bi, hi, pi)
        noise = self._normals(self._row_hash(_TAG_QNOISE, li, bi, hi, pi), w.head_dim)
        u = _uniform(self._row_hash(_TAG_QPICK, li, bi, hi, pi))
        j = torch.clamp((u * pi.to(torch.float64)).to(torch.int64), max=torch.clamp(pi - 1, min=0))
        kj = self._k_raw(li, bi, hi // g, j)
        has_past = (pi > 0).unsqueeze(-1)
        return self._round(torch.where(has_past, 0.5 * kj + noise, noise))


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[name]
