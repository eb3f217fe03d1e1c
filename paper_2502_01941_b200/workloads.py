"""Seeded synthetic inputs for the ShotKV hot path.

This module only *draws inputs*: shot boundaries, K/V/Q tensors and decode-step
vectors.  It holds none of the method's arithmetic (no attention, no scoring,
no selection) and is the one module that both the CUDA tests/bench and the CPU
oracle tests may import.  Tensors are produced with torch on whichever device
is asked for; whoever needs the same bytes on the other side copies them, so
both sides always see identical bf16 values.

The shapes stand in for the paper's workloads (many-shot GSM8K-style prompts of
about 4K tokens and up, long generations of several thousand tokens; Section 4
"Benchmark Design" and the LongGenBench setting).  Only sizes are taken: a
prompt is `S` contiguous shots followed by a question, nothing else.

Recipe
------
* shot lengths: drawn per prompt from the config's distribution, then rescaled
  by largest remainder so that they sum to `N - question_len - preamble`
  exactly, every length clamped to the config's range.
* per (b, l, kv head, shot) an offset vector u ~ N(0, 0.5^2 I_d);
  per (b, l, shot) a relevance rho ~ U[0, 2]; per (b, l) one target shot.
* K[t] = g + rho_s * u_s and V[t] = g' + rho_s * u_s for t in shot s, plain
  N(0,1) rows outside the shots; Qwin[h, w] = g'' + u_{target, h // G}.
  Everything is rounded to bf16 once, at the end.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

BASE_SEED = 20250201


@dataclasses.dataclass(frozen=True)
class PrefillConfig:
    name: str
    B: int
    L: int
    H: int
    Hkv: int
    d: int
    N: int
    W: int
    S: int
    shot_dist: str          # "uniform" | "lognormal"
    shot_lo: int            # uniform: low;  lognormal: clamp low
    shot_hi: int            # uniform: high; lognormal: clamp high
    question_len: int       # tokens after the last shot (includes the window)
    preamble_len: int = 0   # tokens before the first shot
    r_p: float = 0.2
    lognormal_median: float = 300.0
    lognormal_sigma: float = 0.5
    cfg_id: int = 0

    @property
    def G(self) -> int:
        return self.H // self.Hkv

    def replace(self, **kw) -> "PrefillConfig":
        return dataclasses.replace(self, **kw)


# The five workloads of the benchmark plan.  Config 0 is the CPU-seconds case,
# config 3 is the one the headline metric is quoted on.
CONFIGS = {
    0: PrefillConfig("cfg0_tiny", B=1, L=1, H=4, Hkv=2, d=64, N=512, W=16, S=8,
                     shot_dist="uniform", shot_lo=40, shot_hi=70,
                     question_len=-1, r_p=0.4, cfg_id=0),
    1: PrefillConfig("cfg1_llama8b_1layer_4k", B=1, L=1, H=32, Hkv=8, d=128, N=4096, W=32, S=16,
                     shot_dist="uniform", shot_lo=150, shot_hi=300,
                     question_len=200, r_p=0.2, cfg_id=1),
    2: PrefillConfig("cfg2_llama8b_32layer_16k", B=1, L=32, H=32, Hkv=8, d=128, N=16384, W=32, S=48,
                     shot_dist="lognormal", shot_lo=40, shot_hi=1600,
                     question_len=300, r_p=0.2, cfg_id=2),
    3: PrefillConfig("cfg3_llama8b_32layer_32k_b4", B=4, L=32, H=32, Hkv=8, d=128, N=32768, W=64, S=96,
                     shot_dist="uniform", shot_lo=200, shot_hi=480,
                     question_len=500, r_p=0.1, cfg_id=3),
}
CONFIG1_BUDGETS = (0.1, 0.2, 0.4, 0.6, 0.8)


@dataclasses.dataclass(frozen=True)
class DecodeConfig:
    name: str
    B: int
    L: int
    H: int
    Hkv: int
    d: int
    steps: int
    r_d: float
    recompress_every: int
    cfg_id: int = 4

    @property
    def Dcap(self) -> int:
        """Largest decode region ever held: kept entries plus one cycle of appends."""
        R = self.recompress_every
        return int(math.floor(self.r_d * self.steps)) + R


DECODE_CONFIG = DecodeConfig("cfg4_decode_b8", B=8, L=32, H=32, Hkv=8, d=128,
                             steps=1024, r_d=0.25, recompress_every=32)


def _seed(*parts: int) -> int:
    """Mix integers into one 63-bit seed (splitmix-style; order matters)."""
    x = BASE_SEED
    for p in parts:
        x = (x * 6364136223846793005 + 1442695040888963407 + int(p) * 0x9E3779B97F4A7C15) & ((1 << 64) - 1)
        x ^= x >> 31
    return x & ((1 << 63) - 1)


def _largest_remainder(raw: np.ndarray, total: int, lo: int, hi: int) -> np.ndarray:
    """Scale positive `raw` to integers in [lo, hi] that sum to `total`."""
    S = raw.shape[0]
    if not (S * lo <= total <= S * hi):
        raise ValueError(f"cannot fit {S} shots of [{lo},{hi}] tokens into {total}")
    x = raw.astype(np.float64) * (total / raw.sum())
    x = np.clip(x, lo, hi)
    k = np.floor(x).astype(np.int64)
    # hand out / take back the remainder one token at a time, largest fraction first
    order = np.argsort(-(x - k), kind="stable")
    diff = int(total - k.sum())
    i = 0
    guard = 0
    while diff != 0:
        j = order[i % S]
        if diff > 0 and k[j] < hi:
            k[j] += 1
            diff -= 1
        elif diff < 0 and k[j] > lo:
            k[j] -= 1
            diff += 1
        i += 1
        guard += 1
        if guard > 100 * (S + abs(diff) + total):
            raise RuntimeError("largest-remainder rescale did not converge")
    assert k.sum() == total and k.min() >= lo and k.max() <= hi
    return k


def shot_offsets(cfg: PrefillConfig, b: int = 0) -> np.ndarray:
    """Shot boundaries `off[0..S]` (int32) of prompt `b`: shot i is [off[i], off[i+1])."""
    rng = np.random.Generator(np.random.PCG64(_seed(cfg.cfg_id, 101, b, cfg.N, cfg.S)))
    if cfg.shot_dist == "uniform":
        raw = rng.integers(cfg.shot_lo, cfg.shot_hi + 1, size=cfg.S).astype(np.float64)
    elif cfg.shot_dist == "lognormal":
        raw = cfg.lognormal_median * np.exp(cfg.lognormal_sigma * rng.standard_normal(cfg.S))
    else:
        raise ValueError(cfg.shot_dist)
    if cfg.question_len >= 0:
        total = cfg.N - cfg.question_len - cfg.preamble_len
        k = _largest_remainder(raw, total, cfg.shot_lo, cfg.shot_hi)
    else:
        # question = whatever is left after the drawn shots (config 0), at least W tokens
        k = np.clip(np.rint(raw), cfg.shot_lo, cfg.shot_hi).astype(np.int64)
        if cfg.preamble_len + k.sum() > cfg.N - cfg.W:
            k = _largest_remainder(raw, cfg.N - cfg.W - cfg.preamble_len, 1, cfg.shot_hi)
    off = np.empty(cfg.S + 1, dtype=np.int32)
    off[0] = cfg.preamble_len
    off[1:] = cfg.preamble_len + np.cumsum(k)
    assert off[-1] <= cfg.N - cfg.W
    return off


def all_shot_offsets(cfg: PrefillConfig) -> np.ndarray:
    """`[B][S+1]` int32 boundaries, one row per prompt of the batch."""
    return np.stack([shot_offsets(cfg, b) for b in range(cfg.B)], axis=0)


def _gen(device, *parts: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(*parts))
    return g


def prefill_unit(cfg: PrefillConfig, b: int, l: int, off: np.ndarray, device="cpu"):
    """Draw one (prompt b, layer l): Qwin [H,W,d], K [Hkv,N,d], V [Hkv,N,d], all bf16."""
    dev = torch.device(device)
    g = _gen(dev, cfg.cfg_id, 202, b, l)
    Hkv, N, d, S, H, W, G = cfg.Hkv, cfg.N, cfg.d, cfg.S, cfg.H, cfg.W, cfg.G
    u = 0.5 * torch.randn(Hkv, S, d, generator=g, device=dev, dtype=torch.float32)
    rho = 2.0 * torch.rand(S, generator=g, device=dev, dtype=torch.float32)
    target = int(torch.randint(0, S, (1,), generator=g, device=dev).item())
    # shot id of every token; S marks "not in a shot" and indexes a zero row
    shot_id = torch.full((N,), S, dtype=torch.long)
    for i in range(S):
        shot_id[int(off[i]):int(off[i + 1])] = i
    shot_id = shot_id.to(dev)
    shift = torch.cat([u * rho[None, :, None], torch.zeros(Hkv, 1, d, device=dev)], dim=1)  # [Hkv,S+1,d]
    K = torch.randn(Hkv, N, d, generator=g, device=dev, dtype=torch.float32)
    K += shift[:, shot_id, :]
    K = K.to(torch.bfloat16)
    V = torch.randn(Hkv, N, d, generator=g, device=dev, dtype=torch.float32)
    V += shift[:, shot_id, :]
    V = V.to(torch.bfloat16)
    Q = torch.randn(H, W, d, generator=g, device=dev, dtype=torch.float32)
    Q += u[:, target, :].repeat_interleave(G, dim=0)[:, None, :]
    Q = Q.to(torch.bfloat16)
    return Q, K, V


def prefill_batch(cfg: PrefillConfig, device="cpu", offsets: np.ndarray | None = None):
    """Whole workload: Qwin [B,L,H,W,d], K,V [B,L,Hkv,N,d] (bf16) and offsets [B,S+1]."""
    dev = torch.device(device)
    if offsets is None:
        offsets = all_shot_offsets(cfg)
    Q = torch.empty(cfg.B, cfg.L, cfg.H, cfg.W, cfg.d, dtype=torch.bfloat16, device=dev)
    K = torch.empty(cfg.B, cfg.L, cfg.Hkv, cfg.N, cfg.d, dtype=torch.bfloat16, device=dev)
    V = torch.empty_like(K)
    for b in range(cfg.B):
        for l in range(cfg.L):
            q, k, v = prefill_unit(cfg, b, l, offsets[b], dev)
            Q[b, l], K[b, l], V[b, l] = q, k, v
    return Q, K, V, offsets


def decode_step_inputs(cfg: DecodeConfig, step: int, device="cpu"):
    """One decode step: q [B,L,H,d], k_new and v_new [B,L,Hkv,d], all bf16 ~ N(0,1)."""
    dev = torch.device(device)
    g = _gen(dev, cfg.cfg_id, 303, step)
    q = torch.randn(cfg.B, cfg.L, cfg.H, cfg.d, generator=g, device=dev).to(torch.bfloat16)
    k = torch.randn(cfg.B, cfg.L, cfg.Hkv, cfg.d, generator=g, device=dev).to(torch.bfloat16)
    v = torch.randn(cfg.B, cfg.L, cfg.Hkv, cfg.d, generator=g, device=dev).to(torch.bfloat16)
    return q, k, v


def random_prefill_cache(cfg: DecodeConfig, M: int, device="cpu", counts: np.ndarray | None = None):
    """A stand-in compressed prefill region for decode tests: Kc [B,L,Hkv,M,d] bf16 ~ N(0,1)
    and kept_count [B,L] int32 (all M unless `counts` is given)."""
    dev = torch.device(device)
    g = _gen(dev, cfg.cfg_id, 404, M)
    Kc = torch.randn(cfg.B, cfg.L, cfg.Hkv, M, cfg.d, generator=g, device=dev).to(torch.bfloat16)
    if counts is None:
        counts = np.full((cfg.B, cfg.L), M, dtype=np.int32)
    return Kc, torch.from_numpy(np.ascontiguousarray(counts, dtype=np.int32)).to(dev)


def random_prefill_values(cfg: DecodeConfig, M: int, device="cpu") -> torch.Tensor:
    """The values that go with `random_prefill_cache`'s keys: Vc [B,L,Hkv,M,d] bf16 ~ N(0,1)."""
    dev = torch.device(device)
    g = _gen(dev, cfg.cfg_id, 405, M)
    return torch.randn(cfg.B, cfg.L, cfg.Hkv, M, cfg.d, generator=g, device=dev).to(torch.bfloat16)


def bf16_to_f64(x: torch.Tensor) -> np.ndarray:
    """Widen a bf16/f32 tensor to a float64 numpy array (exact)."""
    return x.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def bf16_bits(x: torch.Tensor) -> np.ndarray:
    """The raw 16-bit patterns of a bf16 tensor as a uint16 numpy array."""
    return x.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)
