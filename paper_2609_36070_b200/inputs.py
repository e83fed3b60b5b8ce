"""Seeded synthetic inputs for the MoE layer, shared by the oracle-side tests and the CUDA-side tests.

This module holds none of the method's arithmetic: it only draws numbers, rounds them to the storage
type and names the workload shapes.  Everything is numpy on the host; bf16 tensors are uint16 bit
patterns (round-to-nearest-even from fp32).  The paper's own workload is synthetic N(0,1) data
(Section 4.1), so these inputs do not stand in for any dataset.

Recipe: one Philox stream per tensor (key = (seed, tensor id [, expert id])), `standard_normal(float32)`;
x ~ N(0,1) -> bf16; W_r ~ N(0, 0.02) fp32; expert and shared weights ~ N(0, 0.02) -> bf16;
router bias fp32 per the workload (none / Zipf prior / N(0, 0.5)).
"""
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
import os

import numpy as np

_X, _WR, _BIAS, _WGU, _WD, _SGU, _SD = 1, 2, 3, 4, 5, 6, 7


@dataclass(frozen=True)
class MoEConfig:
    """Shape of one MoE layer workload.  I_s = 0 means no shared expert."""
    name: str
    T: int
    H: int
    E: int
    k: int
    I: int
    I_s: int = 0
    bias: str = "none"        # "none" | "zipf" (b[e] = -1.1 ln(e+1)) | "normal" (b ~ N(0, 0.5))
    seed: int = 0

    @property
    def routes(self) -> int:
        return self.T * self.k

    def ffn_flops(self) -> float:
        """Expert-FFN FLOPs of one forward pass: the paper's 6 N (k+1) D I generalised to I_s != I."""
        return 6.0 * self.T * self.H * (self.k * self.I + self.I_s)

    def with_tokens(self, T: int) -> "MoEConfig":
        return replace(self, T=T, name=f"{self.name}_T{T}")


CONFIGS = {
    "tiny": MoEConfig("tiny", T=256, H=256, E=8, k=2, I=512, I_s=512),
    "qwen3_30b_a3b": MoEConfig("qwen3_30b_a3b", T=16384, H=2048, E=128, k=8, I=768, bias="zipf"),
    "mixtral_8x7b": MoEConfig("mixtral_8x7b", T=8192, H=4096, E=8, k=2, I=14336),
    "gpt_oss_120b": MoEConfig("gpt_oss_120b", T=16384, H=2880, E=128, k=4, I=2880, bias="normal"),
    "deepseek_v3": MoEConfig("deepseek_v3", T=32768, H=7168, E=256, k=8, I=2048, I_s=2048),
}
CONFIG_ORDER = ["tiny", "qwen3_30b_a3b", "mixtral_8x7b", "gpt_oss_120b", "deepseek_v3"]


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round-to-nearest-even.  Finite inputs only."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _rng(seed: int, tensor_id: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64((tensor_id << 32) | sub)]))


def _normal_bf16(seed, tensor_id, sub, shape, std, out=None):
    a = _rng(seed, tensor_id, sub).standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    bits = f32_to_bf16_bits(a)
    if out is not None:
        out[...] = bits
        return out
    return bits


def make_router(cfg: MoEConfig):
    """W_r[E,H] fp32 ~ N(0, 0.02) and the bias[E] fp32 (or None) of the workload."""
    W_r = (_rng(cfg.seed, _WR).standard_normal((cfg.E, cfg.H), dtype=np.float32) * np.float32(0.02)).astype(np.float32)
    if cfg.bias == "none":
        bias = None
    elif cfg.bias == "zipf":
        bias = (-1.1 * np.log(np.arange(1, cfg.E + 1, dtype=np.float64))).astype(np.float32)
    elif cfg.bias == "normal":
        bias = (_rng(cfg.seed, _BIAS).standard_normal((cfg.E,), dtype=np.float32) * np.float32(0.5)).astype(np.float32)
    else:
        raise ValueError(cfg.bias)
    return W_r, bias


def make_x(cfg: MoEConfig) -> np.ndarray:
    """x[T,H] bf16 bits ~ N(0,1).  Drawn in 4096-token blocks so that a shorter T is a prefix of a longer one."""
    out = np.empty((cfg.T, cfg.H), np.uint16)
    for b, t0 in enumerate(range(0, cfg.T, 4096)):
        t1 = min(cfg.T, t0 + 4096)
        blk = _rng(cfg.seed, _X, b).standard_normal((4096, cfg.H), dtype=np.float32)
        out[t0:t1] = f32_to_bf16_bits(blk[: t1 - t0])
    return out


def make_inputs(cfg: MoEConfig, threads: int = 0, experts: bool = True, expert_range=None) -> dict:
    """All tensors of a workload as numpy arrays.

    Keys: x, W_r, bias, W_gate_up [E,2I,H], W_down [E,H,I], W_sgu [2I_s,H] | None, W_sd [H,I_s] | None.
    Expert weights are generated one expert per Philox stream, in a thread pool.  experts=False skips the
    routed expert weights (for routing-only tests); expert_range=(lo, hi) generates only experts lo..hi-1 (the shard
    of one expert-parallel rank: the same values as rows lo..hi-1 of the full tensors).
    """
    W_r, bias = make_router(cfg)
    d = {"x": make_x(cfg), "W_r": W_r, "bias": bias, "W_gate_up": None, "W_down": None,
         "W_sgu": None, "W_sd": None}
    if cfg.I_s > 0:
        d["W_sgu"] = _normal_bf16(cfg.seed, _SGU, 0, (2 * cfg.I_s, cfg.H), 0.02)
        d["W_sd"] = _normal_bf16(cfg.seed, _SD, 0, (cfg.H, cfg.I_s), 0.02)
    if experts:
        lo, hi = expert_range if expert_range is not None else (0, cfg.E)
        Wgu = np.empty((hi - lo, 2 * cfg.I, cfg.H), np.uint16)
        Wd = np.empty((hi - lo, cfg.H, cfg.I), np.uint16)

        def one(e):
            _normal_bf16(cfg.seed, _WGU, e, (2 * cfg.I, cfg.H), 0.02, out=Wgu[e - lo])
            _normal_bf16(cfg.seed, _WD, e, (cfg.H, cfg.I), 0.02, out=Wd[e - lo])

        n = threads or min(32, os.cpu_count() or 1)
        if n > 1 and hi - lo > 1:
            with ThreadPoolExecutor(n) as ex:
                list(ex.map(one, range(lo, hi)))
        else:
            for e in range(lo, hi):
                one(e)
        d["W_gate_up"], d["W_down"] = Wgu, Wd
    return d


def sample_tokens(cfg: MoEConfig, idx: np.ndarray, n: int, seed: int = 1) -> np.ndarray:
    """Token sample for spot checks at full size: the first min(128, n) tokens, then random ones,
    extended until every expert that owns a route also owns a sampled route.  Sorted, unique."""
    T = idx.shape[0]
    n = min(n, T)
    rng = np.random.Generator(np.random.Philox(key=[np.uint64(cfg.seed), np.uint64(0xABCD0000 + seed)]))
    head = np.arange(min(128, n))
    rest = rng.permutation(np.arange(head.size, T))
    chosen = list(head) + list(rest[: n - head.size])
    covered = np.zeros(cfg.E, bool)
    covered[np.unique(idx[chosen])] = True
    used = np.zeros(cfg.E, bool)
    used[np.unique(idx)] = True
    if not covered[used].all():
        for t in rest[n - head.size:]:
            if (~covered[idx[t]]).any():
                chosen.append(int(t))
                covered[idx[t]] = True
                if covered[used].all():
                    break
    return np.unique(np.asarray(chosen, np.int32))
