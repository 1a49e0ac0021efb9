"""Seeded synthetic inputs for the verify-and-feedback step.

This module only makes inputs: logits with the shapes and value structure of the workloads
(vocabulary sizes of the Vicuna/Llama-2 and Qwen3 families and a 128 256-entry vocabulary,
k = 4..8 draft tokens, fp32 or bf16), draft tokens drawn from the draft distribution (the
"Generate the draft sequence" step of Algorithm 1, which happens before the path built here),
and the pre-drawn uniforms.  It contains none of the verification arithmetic and is used by the
tests, the benchmark and the smoke check to feed the same bytes to the CUDA path and to the CPU
oracle.  Everything is numpy on the host.

Randomness is counter-based (Philox) and keyed by (seed, config, sequence), so any sequence of
any config can be regenerated on its own and in any order.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Dict, Optional, Sequence

import numpy as np

BASE_SEED = 20260312


@dataclass(frozen=True)
class Config:
    """One synthetic workload.  ``recipe`` selects the value structure below."""
    name: str
    B: int
    k: int
    V: int
    dtype: str          # "f32" or "bf16"
    tau: float
    recipe: str         # "gauss", "peaks", "zipf", "zipf_mixed"
    t_sigma: float      # std of the Gaussian body of the target logits
    d_sigma: float      # std of the draft noise (ignored by "zipf_mixed")
    d_scale: float = 1.0    # draft = d_scale * target + noise
    zipf_s: float = 0.0     # exponent of the Zipf log-prior
    index: int = 0

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def algorithmic_bytes(self) -> int:
        """Read (2k+1)*V*B logits, write k*V*B gradient entries."""
        return ((2 * self.k + 1) + self.k) * self.V * self.B * self.elem_bytes

    def with_batch(self, B: int) -> "Config":
        return Config(**{**self.__dict__, "B": B})


CONFIGS: Dict[str, Config] = {c.name: c for c in [
    Config("cfg1", B=1, k=4, V=32000, dtype="f32", tau=1.0, recipe="gauss",
           t_sigma=2.0, d_sigma=0.5, index=1),
    Config("cfg2", B=8, k=5, V=32000, dtype="bf16", tau=0.7, recipe="peaks",
           t_sigma=3.0, d_sigma=1.0, index=2),
    Config("cfg3", B=32, k=8, V=128256, dtype="bf16", tau=1.0, recipe="zipf",
           t_sigma=2.5, d_sigma=1.5, d_scale=0.8, zipf_s=1.1, index=3),
    Config("cfg4", B=64, k=4, V=151936, dtype="bf16", tau=0.8, recipe="zipf_mixed",
           t_sigma=2.0, d_sigma=0.0, zipf_s=1.0, index=4),
    Config("cfg5", B=256, k=6, V=128256, dtype="f32", tau=1.0, recipe="gauss",
           t_sigma=2.0, d_sigma=0.8, index=5),
]}


@dataclass
class Inputs:
    cfg: Config
    target_logits: np.ndarray   # [B,k+1,V] float32, or uint16 holding bf16 bits
    draft_logits: np.ndarray    # [B,k,V]
    draft_tokens: np.ndarray    # [B,k] int32
    uniforms: np.ndarray        # [B,k+1] float32 in [0,1)
    tau: float
    seed: int


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns the 16-bit patterns."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = bits + (np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float32."""
    return (np.ascontiguousarray(a, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, cfg_index: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed + cfg_index) & (2**64 - 1), stream]))


def _uniform24(rng: np.random.Generator, n: int) -> np.ndarray:
    """fp32 uniforms in [0,1): 24 random bits over 2**24."""
    return (rng.integers(0, 1 << 24, size=n, dtype=np.uint32).astype(np.float32)
            / np.float32(16777216.0))


def _vocab_prior(cfg: Config, seed: int) -> Optional[np.ndarray]:
    """Zipf log-prior -s*ln(rank) over one random permutation of the vocabulary."""
    if cfg.zipf_s == 0.0:
        return None
    rng = _rng(seed, cfg.index, 2**63)
    rank = rng.permutation(cfg.V).astype(np.float64) + 1.0
    return -cfg.zipf_s * np.log(rank)


def _one_sequence(cfg: Config, seed: int, b: int, prior: Optional[np.ndarray]):
    rng = _rng(seed, cfg.index, b)
    k, V = cfg.k, cfg.V
    T = rng.standard_normal((k + 1, V)) * cfg.t_sigma
    if cfg.recipe == "peaks":
        for i in range(k + 1):
            idx = rng.choice(V, size=min(50, V), replace=False)
            T[i, idx] += 8.0
    if prior is not None:
        T += prior[None, :]
    if cfg.recipe == "zipf_mixed":
        sigma = rng.uniform(0.2, 3.0)
    else:
        sigma = cfg.d_sigma
    D = cfg.d_scale * T[:k] + rng.standard_normal((k, V)) * sigma
    T32 = T.astype(np.float32)
    D32 = D.astype(np.float32)
    if cfg.dtype == "bf16":
        T_out = f32_to_bf16_bits(T32)
        D_out = f32_to_bf16_bits(D32)
        D_val = bf16_bits_to_f32(D_out).astype(np.float64)
    else:
        T_out, D_out = T32, D32
        D_val = D32.astype(np.float64)
    # draft tokens: inverse-CDF draw from softmax(D/tau) of the logits as delivered
    z = D_val / cfg.tau
    z -= z.max(axis=1, keepdims=True)
    e = np.exp(z)
    cdf = np.cumsum(e, axis=1)
    w = rng.random(k) * cdf[:, -1]
    x = np.array([min(int(np.searchsorted(cdf[i], w[i], side="right")), V - 1) for i in range(k)],
                 dtype=np.int32)
    u = _uniform24(rng, k + 1)
    return T_out, D_out, x, u


def make_inputs(cfg: Config, seed: int = BASE_SEED, sequences: Optional[Sequence[int]] = None,
                workers: int = 8) -> Inputs:
    """Inputs for ``cfg``; ``sequences`` picks a subset of sequence indices (default: all B)."""
    seqs = list(range(cfg.B)) if sequences is None else [int(b) for b in sequences]
    n = len(seqs)
    np_dtype = np.float32 if cfg.dtype == "f32" else np.uint16
    T = np.empty((n, cfg.k + 1, cfg.V), np_dtype)
    D = np.empty((n, cfg.k, cfg.V), np_dtype)
    x = np.empty((n, cfg.k), np.int32)
    u = np.empty((n, cfg.k + 1), np.float32)
    prior = _vocab_prior(cfg, seed)

    def work(j):
        T[j], D[j], x[j], u[j] = _one_sequence(cfg, seed, seqs[j], prior)

    if n > 1 and workers > 1:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(work, range(n)))
    else:
        for j in range(n):
            work(j)
    return Inputs(cfg=cfg, target_logits=T, draft_logits=D, draft_tokens=x, uniforms=u,
                  tau=cfg.tau, seed=seed)


def custom_config(B: int, k: int, V: int, dtype: str = "f32", tau: float = 1.0,
                  recipe: str = "gauss", t_sigma: float = 2.0, d_sigma: float = 0.7,
                  d_scale: float = 1.0, zipf_s: float = 0.0, index: int = 99) -> Config:
    """A free-form workload for edge-case tests (odd V, k = 1, ...)."""
    return Config(f"custom_B{B}_k{k}_V{V}_{dtype}", B=B, k=k, V=V, dtype=dtype, tau=tau,
                  recipe=recipe, t_sigma=t_sigma, d_sigma=d_sigma, d_scale=d_scale, zipf_s=zipf_s,
                  index=index)


def ensemble_drafts(inp: Inputs, n_learners: int, seed: int = BASE_SEED) -> list:
    """Draft logits of ``n_learners`` base learners for the inputs of one round: learner 0 is the
    workload's own draft, learner n > 0 is the target's rows plus Gaussian noise whose standard
    deviation doubles from learner to learner (base learners that track the target ever more
    loosely, like draft heads trained with ever larger step sizes).  Same dtype as the inputs."""
    cfg = inp.cfg
    k = cfg.k
    T = inp.target_logits[:, :k]
    Tf = bf16_bits_to_f32(T) if cfg.dtype == "bf16" else T
    out = [inp.draft_logits]
    sigma0 = cfg.d_sigma if cfg.d_sigma > 0 else 0.5
    for n in range(1, n_learners):
        rng = _rng(seed, cfg.index, 1000 + n)
        noise = rng.standard_normal(Tf.shape, dtype=np.float32) * np.float32(sigma0 * 2.0 ** n)
        D = Tf + noise
        out.append(f32_to_bf16_bits(D) if cfg.dtype == "bf16" else D.astype(np.float32))
    return out


def lmhead_operands(R: int, V: int, d: int, seed: int = BASE_SEED):
    """Operands of the output layer's gradient dW = g^T X as bf16 bit patterns: g [R,V] shaped like a
    gradient with respect to logits (most entries tiny, a few large per row), X [R,d] ~ N(0,1)."""
    rng = np.random.Generator(np.random.Philox(key=[seed & (2**64 - 1), 77]))
    g = rng.standard_normal((R, V), dtype=np.float32) * np.float32(1e-3)
    hot = rng.integers(0, V, (R, 3))
    g[np.arange(R)[:, None], hot] += rng.standard_normal((R, 3), dtype=np.float32) * np.float32(0.3)
    X = rng.standard_normal((R, d), dtype=np.float32)
    return f32_to_bf16_bits(g), f32_to_bf16_bits(X)
