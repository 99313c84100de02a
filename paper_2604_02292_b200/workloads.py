"""Seeded synthetic inputs for the HCCS kernels and for their CPU oracle.

This module only draws numbers (NumPy ``Generator(PCG64(seed))``); it holds
none of the method's arithmetic and imports neither the CUDA binding nor the
oracle, so that both sides can be fed the same bytes.

The five named workloads stand in for the int8 attention logits of small
encoder models at 64 and 128 keys (the shapes of the paper's evaluation) and a
BERT-base-like 512-key shape; no dataset or trained weight is involved.

Draw order inside one workload (fixed, so a workload is reproducible from its
seed alone): per-head logit scales, then per-head theta = (B, S, Dmax), then the
per-head requantisation multipliers (fused workload only), then the data in
blocks of whole batch entries in row-major order, then the dominant-logit
choices (workload 2 only).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SEED_BASE = 260402292 * 10

# Mode flags of the public API (kept equal to include/hccs.h; restated here so
# that this module needs nothing but numpy).
FLAG_OUT_U16 = 1
FLAG_RECIP_CLB = 2
FLAG_CAUSAL = 4


@dataclass
class Workload:
    name: str
    shape: tuple                      # (B, H, Lq, Lk) for standalone; (B, H, L, d) for fused
    flags: int
    n_design: int
    theta: np.ndarray                 # int32 [H, 3] = (B_h, S_h, Dmax_h)
    logits: np.ndarray | None = None  # int8 [B, H, Lq, Lk]
    Q: np.ndarray | None = None       # fused: int8 [B, H, L, d]
    K: np.ndarray | None = None
    V: np.ndarray | None = None
    requant_mult: np.ndarray | None = None   # fused: int32 [H]
    requant_shift: int = 20
    meta: dict = field(default_factory=dict)

    @property
    def rows(self) -> int:
        return int(self.shape[0] * self.shape[1] * self.shape[2])

    @property
    def elements(self) -> int:
        if self.logits is not None:
            return int(self.logits.size)
        b, h, l, _ = self.shape
        return int(b * h * l * l)


def band(n: int):
    """(floor score, largest B) of the admissible band for B_h at row length n (Eq. 11)."""
    return -(-256 // n), 32767 // n


def sample_theta(rng: np.random.Generator, H: int, n: int) -> np.ndarray:
    """Per-head (B, S, Dmax) drawn uniformly inside the band of Eq. 11 for length n."""
    f, bmax = band(n)
    room = bmax - f
    if room < 0:
        raise ValueError(f"no admissible B_h for n={n}")
    out = np.zeros((H, 3), dtype=np.int32)
    for h in range(H):
        d_hi = max(1, min(127, room))
        d_lo = min(4, d_hi)
        D = int(rng.integers(d_lo, d_hi + 1))
        s_hi = min(127, room // D)
        s_lo = min(1, s_hi)
        S = int(rng.integers(s_lo, s_hi + 1))
        B = int(rng.integers(S * D + f, bmax + 1))
        out[h] = (B, S, D)
    return out


def _clip_round_i8(a: np.ndarray) -> np.ndarray:
    return np.clip(np.rint(a), -128, 127).astype(np.int8)


def gaussian_logits(rng, shape, sigma_h, block_batches: int = 64) -> np.ndarray:
    """clip(round(N(0, sigma_h)), -128, 127) per head, drawn in blocks of batch entries."""
    Bt, H, Lq, Lk = shape
    out = np.empty(shape, dtype=np.int8)
    sig = np.asarray(sigma_h, dtype=np.float32).reshape(1, H, 1, 1)
    for b0 in range(0, Bt, block_batches):
        b1 = min(Bt, b0 + block_batches)
        z = rng.standard_normal((b1 - b0, H, Lq, Lk), dtype=np.float32)
        out[b0:b1] = _clip_round_i8(z * sig)
    return out


def laplace_logits(rng, shape, scale_h, block_batches: int = 4) -> np.ndarray:
    """clip(round(Laplace(0, b_h)), -128, 127) per head (heavy-tailed logits)."""
    Bt, H, Lq, Lk = shape
    out = np.empty(shape, dtype=np.int8)
    sc = np.asarray(scale_h, dtype=np.float64).reshape(1, H, 1, 1)
    for b0 in range(0, Bt, block_batches):
        b1 = min(Bt, b0 + block_batches)
        z = rng.laplace(0.0, 1.0, size=(b1 - b0, H, Lq, Lk))
        out[b0:b1] = _clip_round_i8(z * sc)
    return out


def add_dominant_logits(rng, logits: np.ndarray, fraction: float = 0.05, boost: int = 100):
    """Give a seeded ``fraction`` of rows one dominant logit: clip(round(row mean) + boost)."""
    Bt, H, Lq, Lk = logits.shape
    rows = Bt * H * Lq
    flat = logits.reshape(rows, Lk)
    k = int(round(rows * fraction))
    chosen = rng.choice(rows, size=k, replace=False)
    cols = rng.integers(0, Lk, size=k)
    means = np.rint(flat[chosen].astype(np.float64).mean(axis=1))
    flat[chosen, cols] = np.clip(means + boost, -128, 127).astype(np.int8)
    return np.sort(chosen)


def make_config(c: int, batch: int | None = None) -> Workload:
    """Workload ``c`` in 1..5.  ``batch`` overrides the batch size (same recipe, same
    per-head draws; the data stream is then a prefix in batch order)."""
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + c))
    if c == 1 or c == 2:
        H, Lq, Lk = 4, 64, 64
        Bt = (1 if c == 1 else 4096) if batch is None else batch
        sigma = rng.uniform(8.0, 40.0, size=H)
        theta = sample_theta(rng, H, Lk)
        x = gaussian_logits(rng, (Bt, H, Lq, Lk), sigma)
        meta = {"sigma_h": sigma.tolist()}
        if c == 2:
            meta["dominant_rows"] = int(add_dominant_logits(rng, x).size)
        return Workload(f"config{c}", (Bt, H, Lq, Lk), 0, Lk, theta, logits=x, meta=meta)
    if c == 3:
        H, Lq, Lk = 8, 128, 128
        Bt = 256 if batch is None else batch
        sigma = rng.uniform(4.0, 60.0, size=H)
        theta = sample_theta(rng, H, Lk)
        x = gaussian_logits(rng, (Bt, H, Lq, Lk), sigma)
        return Workload("config3", (Bt, H, Lq, Lk), FLAG_CAUSAL, Lk, theta, logits=x,
                        meta={"sigma_h": sigma.tolist()})
    if c == 4:
        H, Lq, Lk = 12, 512, 512
        Bt = 64 if batch is None else batch
        scale = rng.uniform(6.0, 30.0, size=H)
        theta = sample_theta(rng, H, Lk)
        x = laplace_logits(rng, (Bt, H, Lq, Lk), scale)
        return Workload("config4", (Bt, H, Lq, Lk), 0, Lk, theta, logits=x,
                        meta={"laplace_scale_h": scale.tolist()})
    if c == 5:
        H, L, d = 12, 1024, 64
        Bt = 32 if batch is None else batch
        theta = sample_theta(rng, H, L)
        mult = rng.integers(768, 3841, size=H).astype(np.int32)
        Q = rng.integers(-64, 64, size=(Bt, H, L, d), dtype=np.int8)
        K = rng.integers(-64, 64, size=(Bt, H, L, d), dtype=np.int8)
        V = rng.integers(-64, 64, size=(Bt, H, L, d), dtype=np.int8)
        return Workload("config5", (Bt, H, L, d), 0, L, theta, Q=Q, K=K, V=V,
                        requant_mult=mult, requant_shift=20)
    raise ValueError("config index must be 1..5")


def make_attention(seed: int, shape) -> Workload:
    """Fused-attention operands of any [B, H, L, d], drawn like workload 5's: uniform int8 in
    [-64, 63], theta in the band for L keys, multipliers scaled by 64 / d so that the logits keep
    workload 5's spread."""
    Bt, H, L, d = (int(v) for v in shape)
    rng = np.random.Generator(np.random.PCG64(int(seed)))
    theta = sample_theta(rng, H, L)
    mult = (rng.integers(768, 3841, size=H) * 64 // d).astype(np.int32)
    Q, K, V = (rng.integers(-64, 64, size=(Bt, H, L, d), dtype=np.int8) for _ in range(3))
    return Workload("attention" + "x".join(str(v) for v in (Bt, H, L, d)), (Bt, H, L, d), 0, L, theta,
                    Q=Q, K=K, V=V, requant_mult=mult, requant_shift=20)


def make_rows(seed: int, shape, n_design: int | None = None, kind: str = "gauss",
              flags: int = 0) -> Workload:
    """Small seeded standalone workload of any shape, for parity and edge-case tests.

    kind: "gauss" (sigma_h ~ U[4,60]), "laplace" (b_h ~ U[6,30]), "uniform" (all of
    int8), "const" (one value per row), "extreme" (only -128 / 127).
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    Bt, H, Lq, Lk = shape
    n = Lk if n_design is None else n_design
    theta = sample_theta(rng, H, max(n, 1))
    if Bt * H * Lq * Lk == 0:
        x = np.zeros(shape, dtype=np.int8)
    elif kind == "gauss":
        x = gaussian_logits(rng, shape, rng.uniform(4.0, 60.0, size=H))
    elif kind == "laplace":
        x = laplace_logits(rng, shape, rng.uniform(6.0, 30.0, size=H))
    elif kind == "uniform":
        x = rng.integers(-128, 128, size=shape, dtype=np.int8)
    elif kind == "const":
        x = np.broadcast_to(rng.integers(-128, 128, size=(Bt, H, Lq, 1), dtype=np.int8),
                            shape).copy()
    elif kind == "extreme":
        x = np.where(rng.random(shape) < 0.5, -128, 127).astype(np.int8)
    else:
        raise ValueError(kind)
    return Workload(f"rows-{kind}-{seed}", tuple(shape), flags, n, theta, logits=x)


def shard_rows(total_rows: int, world_size: int, rank: int, granule: int = 1):
    """Contiguous row range [r0, r1) owned by ``rank``: rows are independent, so the
    path shards with no exchange.  Boundaries fall on multiples of ``granule`` rows."""
    units = -(-total_rows // granule)
    u0 = (units * rank) // world_size
    u1 = (units * (rank + 1)) // world_size
    return min(total_rows, u0 * granule), min(total_rows, u1 * granule)
