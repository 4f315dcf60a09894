"""Seeded synthetic inputs shared by the CUDA tests, the benchmark and the CPU oracle's tests.

This module only draws random tensors and describes workload shapes.  It holds
none of the method's arithmetic (no nugget counts, no scores, no selection, no
attention) so that the CUDA path and the oracle stay independent of each other.

The paper evaluates on text corpora with LLaMA weights; neither is available
offline, so tensors with the same shapes and simple Gaussian statistics stand in
for them: hidden states ~ N(0, 1), Scorer weights ~ N(0, 1/d), projection
weights ~ N(0, 1/d), and for the LLaMA-sized workloads Q, K, V ~ N(0, 1) drawn
directly.  Every tensor is drawn in fp32 from a generator seeded by a hash of
its tags and cast once to the storage dtype; the cast tensor is the ground
truth for every consumer.
"""
from __future__ import annotations

import hashlib
import math
from dataclasses import dataclass, field

import numpy as np
import torch


def seed_for(*tags) -> int:
    """Stable 63-bit seed from arbitrary tags (ints, strings)."""
    h = hashlib.sha256(repr(tags).encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 63) - 1)


def randn(shape, *tags, std: float = 1.0, dtype=torch.float32, device="cpu") -> torch.Tensor:
    """N(0, std^2) tensor drawn in fp32 on ``device`` from a tag-seeded generator, cast to ``dtype``.

    CPU and CUDA generators produce different streams: consumers that must see
    the same values draw on one device and copy.
    """
    g = torch.Generator(device=device)
    g.manual_seed(seed_for(*tags))
    t = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        t.mul_(std)
    return t.to(dtype)


def to_numpy(t: torch.Tensor) -> np.ndarray:
    """Host numpy view of a tensor in its storage format (bf16 -> uint16 bit patterns)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def offsets(lengths) -> np.ndarray:
    """Exclusive prefix sums as int32[B+1]."""
    out = np.zeros(len(lengths) + 1, dtype=np.int32)
    np.cumsum(np.asarray(lengths, dtype=np.int64), out=out[1:])
    return out


def loguniform_lengths(B: int, lo: int, hi: int, *tags) -> list[int]:
    """B integer lengths, log-uniform in [lo, hi]."""
    rs = np.random.RandomState(seed_for(*tags) % (2 ** 32))
    u = rs.uniform(math.log(lo), math.log(hi), size=B)
    return [int(min(hi, max(lo, round(math.exp(x))))) for x in u]


def project(X: torch.Tensor, W: torch.Tensor) -> torch.Tensor:
    """Input synthesis for the small fp32 workload: X @ W in fp64, rounded once to X's dtype."""
    return (X.double() @ W.double()).to(X.dtype)


def stress_scores(kind: str, n: int, *tags) -> np.ndarray:
    """fp32 score vectors that exercise ties and special values in TopK.

    Trained Scorers concentrate on a few delimiter token types (Sec. 4.3), so
    near-duplicate scores are the realistic hard case.
    """
    rs = np.random.RandomState(seed_for(kind, n, *tags) % (2 ** 32))
    if kind == "normal":
        s = rs.standard_normal(n)
    elif kind == "quantised8":
        s = rs.randint(0, 8, size=n) * 0.25 - 1.0
    elif kind == "two_valued":
        s = rs.randint(0, 2, size=n).astype(np.float64)
    elif kind == "all_equal":
        s = np.full(n, 0.5)
    elif kind == "ascending":
        s = np.arange(n, dtype=np.float64)
    elif kind == "descending":
        s = -np.arange(n, dtype=np.float64)
    elif kind == "signed_zeros":
        s = np.where(rs.randint(0, 2, size=n) == 0, 0.0, -0.0)
    elif kind == "specials":
        s = rs.standard_normal(n)
        pick = rs.randint(0, 6, size=n)
        s = np.where(pick == 0, np.inf, s)
        s = np.where(pick == 1, -np.inf, s)
        s = np.where(pick == 2, np.nan, s)
        s = np.where(pick == 3, 0.0, s)
        s = np.where(pick == 4, -0.0, s)
    elif kind == "denormals":
        s = rs.randint(-4, 5, size=n).astype(np.float64) * 1e-45
    else:
        raise ValueError(kind)
    return s.astype(np.float32)


STRESS_KINDS = ("normal", "quantised8", "two_valued", "all_equal", "ascending", "descending",
                "signed_zeros", "specials", "denormals")


@dataclass(frozen=True)
class Workload:
    """Shape of one benchmark/parity configuration (no derived method quantities)."""
    name: str
    dtype: torch.dtype
    n_ctx: tuple            # compressed-context length per sequence
    d: int
    H: int
    dh: int
    ratios: tuple = (10,)   # compression ratios r
    local: int = 0          # uncompressed context tokens kept beside the nuggets
    tq_dense: int = 0       # size of the dense query block (0 = none)
    decode_steps: int = 0
    layers: int = 1
    project_kv: bool = False  # K = X W_K, V = X W_V with W ~ N(0, 1/d) instead of K, V ~ N(0, 1)
    note: str = ""

    @property
    def B(self) -> int:
        return len(self.n_ctx)


def _c5_lengths():
    return tuple(loguniform_lengths(64, 512, 32768, "config5", "lengths"))


WORKLOADS = {
    # Tiny fp32 single layer: 16 query tokens attend 52 nuggets and, causally, themselves.
    "c1_tiny_fp32": Workload("c1_tiny_fp32", torch.float32, (512,), 256, 4, 64,
                             tq_dense=16, project_kv=True),
    # LLaMA-7B-shaped single layer: all 2048 context tokens compressed, 64 more uncompressed
    # tokens seed a local window that slides with each of the 128 decode tokens.
    "c2_llama7b_decode": Workload("c2_llama7b_decode", torch.bfloat16, (2048,) * 8, 4096, 32, 128,
                                  local=64, decode_steps=128),
    # LLaMA-7B-shaped AR mode, 32 independent layers: 7168 compressed + 1024 uncompressed,
    # a 256-token query block, then 64 decode tokens.
    "c3_llama7b_ar": Workload("c3_llama7b_ar", torch.bfloat16, (7168,) * 4, 4096, 32, 128,
                              local=1024, tq_dense=256, decode_steps=64, layers=32),
    # LLaMA-13B-shaped ratio sweep.
    "c4_llama13b_sweep": Workload("c4_llama13b_sweep", torch.bfloat16, (16384,), 5120, 40, 128,
                                  ratios=(1, 5, 10, 20), tq_dense=512, decode_steps=128, layers=40),
    # Ragged serving batch.
    "c5_ragged_serving": Workload("c5_ragged_serving", torch.bfloat16, _c5_lengths(), 4096, 32, 128,
                                  decode_steps=256, layers=32,
                                  note="segment append: every 64 decoded tokens are compressed"),
}
