"""Seeded synthetic workloads: the five frozen configurations and their input generators.

This module holds no arithmetic of the method.  It only draws numbers: length vectors
(frozen as literals so no RNG-version dependence remains), token features, and weights.
Both the CPU oracle's tests and the CUDA path's tests/benchmarks take their inputs from
here, so the two sides always see identical arrays.

Conventions (the readings are listed in the design notes of the repository):
  * weights are ``[out, in]`` row-major and drawn as ``xi / sqrt(fan_in)`` with xi ~ N(0,1)
    ("N(0, 1/fan_in)" read as a variance);
  * LayerNorm scale ``gamma = 1 + 0.1 xi`` and shift ``beta = 0.1 xi'`` so the affine part is exercised;
  * no linear biases anywhere;
  * for the bf16 configurations every array is rounded once to bf16 (round to nearest even)
    and handed out as float32 holding exactly representable bf16 values.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List

import numpy as np


@dataclass(frozen=True)
class Config:
    name: str
    dtype: str          # "f32" or "bf16" (storage type of inputs/weights/intermediates)
    lengths: tuple      # frozen per-sample lengths N_s
    c_s: int            # token (single) width
    c_z: int            # pair width (config 4: the token hidden width the attention runs on)
    c_h: int            # triangle hidden width
    H: int              # attention heads
    d: int              # head dim
    blocks: int         # stacked blocks
    seed: int
    kind: str = "pair"  # "pair": full Pairformer-style block; "token": single-ragged special case

    @property
    def B(self) -> int:
        return len(self.lengths)

    @property
    def T1(self) -> int:
        return int(sum(self.lengths))

    @property
    def T2(self) -> int:
        return int(sum(n * n for n in self.lengths))

    @property
    def N3(self) -> int:
        return int(sum(n ** 3 for n in self.lengths))

    @property
    def N_max(self) -> int:
        return int(max(self.lengths)) if self.lengths else 0


# Length vectors were drawn once (NumPy default_rng, seeds 2, 3, 4 with the laws named in each
# comment) and are frozen here as literals.
CONFIGS: Dict[str, Config] = {
    # tiny correctness block, fp32
    "cfg1": Config("cfg1", "f32", (5, 9, 13, 16), c_s=32, c_z=16, c_h=16, H=2, d=8, blocks=1, seed=1001),
    # near-uniform lengths: uniform integers in [208, 224]
    "cfg2": Config("cfg2", "bf16", (222, 212, 209, 213, 215, 221, 215, 209),
                   c_s=384, c_z=128, c_h=128, H=4, d=32, blocks=4, seed=1002),
    # high variation: log-uniform 32..768
    "cfg3": Config("cfg3", "bf16", (42, 68, 408, 204, 43, 127, 147, 53, 330, 46, 111, 165, 126, 207, 334, 668),
                   c_s=384, c_z=128, c_h=128, H=4, d=32, blocks=4, seed=1003),
    # single-ragged token-axis special case: lognormal(5.2, 0.6) clipped to [16, 512]
    "cfg4": Config("cfg4", "bf16", (123, 163, 492, 269, 68, 181, 125, 198, 69, 210, 209, 467, 219, 246, 74, 512,
                                    57, 351, 149, 107, 122, 121, 228, 170, 441, 60, 181, 106, 289, 51, 147, 206),
                   c_s=768, c_z=768, c_h=0, H=12, d=64, blocks=1, seed=1004, kind="token"),
    # large pair-state stress
    "cfg5": Config("cfg5", "bf16", (384, 1024, 1536, 2048), c_s=256, c_z=64, c_h=64, H=4, d=16, blocks=2, seed=1005),
}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round a float32 array to the nearest bf16 (ties to even); result is float32 with the
    low 16 mantissa bits zero.  NaN/Inf do not occur in these workloads."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of an array already holding bf16-representable float32 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


class _Stream:
    def __init__(self, seed: int, bf16: bool):
        self.rng = np.random.default_rng(seed)
        self.bf16 = bf16

    def _fin(self, a):
        a = a.astype(np.float32)
        return round_to_bf16(a) if self.bf16 else a

    def normal(self, *shape):
        return self._fin(self.rng.standard_normal(shape, dtype=np.float32))

    def weight(self, out_f: int, in_f: int):
        return self._fin(self.rng.standard_normal((out_f, in_f), dtype=np.float32) / np.float32(np.sqrt(in_f)))

    def ln_gamma(self, c: int):
        return self._fin(1.0 + 0.1 * self.rng.standard_normal(c, dtype=np.float32))

    def ln_beta(self, c: int):
        return self._fin(0.1 * self.rng.standard_normal(c, dtype=np.float32))


def make_block_weights(st: _Stream, cfg: Config) -> dict:
    """Weights of one Pairformer-style block, drawn in call order."""
    c_s, c_z, c_h, Hd = cfg.c_s, cfg.c_z, cfg.c_h, cfg.H * cfg.d
    w = {}
    w["broadcast"] = dict(W_a=st.weight(c_z, c_s), W_b=st.weight(c_z, c_s),
                          ln_gamma=st.ln_gamma(c_z), ln_beta=st.ln_beta(c_z))
    w["trimul"] = dict(ln_in_gamma=st.ln_gamma(c_z), ln_in_beta=st.ln_beta(c_z),
                       W_ap=st.weight(c_h, c_z), W_ag=st.weight(c_h, c_z),
                       W_bp=st.weight(c_h, c_z), W_bg=st.weight(c_h, c_z),
                       W_g=st.weight(c_z, c_z),
                       ln_out_gamma=st.ln_gamma(c_h), ln_out_beta=st.ln_beta(c_h),
                       W_o=st.weight(c_z, c_h))
    w["attn"] = dict(ln_gamma=st.ln_gamma(c_z), ln_beta=st.ln_beta(c_z),
                     W_q=st.weight(Hd, c_z), W_k=st.weight(Hd, c_z), W_v=st.weight(Hd, c_z),
                     W_b=st.weight(cfg.H, c_z), W_g=st.weight(Hd, c_z), W_o=st.weight(c_z, Hd))
    w["reduce"] = dict(W_r=st.weight(c_s, c_z))
    return w


def make_transition_weights(cfg: Config, block: int = 0, expansion: int = 4) -> dict:
    """Weights of the SwiGLU pair transition of one block (hidden = expansion * c_z).  They come from a stream of
    their own (seed + 7919 * (block + 1)), so the frozen draws of the other sub-layers are unchanged."""
    st = _Stream(cfg.seed + 7919 * (block + 1), cfg.dtype == "bf16")
    c, hid = cfg.c_z, expansion * cfg.c_z
    return dict(ln_gamma=st.ln_gamma(c), ln_beta=st.ln_beta(c), W_a=st.weight(hid, c), W_b=st.weight(hid, c),
                W_2=st.weight(c, hid))


def make_single_attn_weights(cfg: Config, block: int = 0) -> dict:
    """Weights of the pair-biased single attention of one block (tokens of width c_s, bias from the pair state of
    width c_z, H heads of d).  A stream of its own (seed + 104729 * (block + 1)): the frozen draws are unchanged."""
    st = _Stream(cfg.seed + 104729 * (block + 1), cfg.dtype == "bf16")
    c, cz, Hd = cfg.c_s, cfg.c_z, cfg.H * cfg.d
    return dict(ln_gamma=st.ln_gamma(c), ln_beta=st.ln_beta(c), W_q=st.weight(Hd, c), W_k=st.weight(Hd, c),
                W_v=st.weight(Hd, c), W_g=st.weight(Hd, c), W_o=st.weight(c, Hd),
                ln_z_gamma=st.ln_gamma(cz), ln_z_beta=st.ln_beta(cz), W_b=st.weight(cfg.H, cz))


def make_token_weights(st: _Stream, cfg: Config) -> dict:
    """Weights of the single-ragged special case: attention over the token axis, no LN/gate/bias."""
    c, Hd = cfg.c_z, cfg.H * cfg.d
    return dict(W_q=st.weight(Hd, c), W_k=st.weight(Hd, c), W_v=st.weight(Hd, c), W_o=st.weight(c, Hd))


def make_inputs(cfg: Config, lengths=None) -> dict:
    """All arrays of one configuration: ``x`` [T1, c_s] and a list of per-block weight dicts.
    ``lengths`` may override the frozen vector (used by invariance tests); the draw order is
    x first, then per block the weights in call order."""
    lengths = tuple(cfg.lengths if lengths is None else lengths)
    st = _Stream(cfg.seed, cfg.dtype == "bf16")
    T1 = int(sum(lengths))
    x = st.normal(T1, cfg.c_s)
    if cfg.kind == "token":
        blocks = [make_token_weights(st, cfg) for _ in range(cfg.blocks)]
    else:
        blocks = [make_block_weights(st, cfg) for _ in range(cfg.blocks)]
    return dict(lengths=np.asarray(lengths, dtype=np.int64), x=x, blocks=blocks)


def pair_occupancy(lengths) -> float:
    """rho_pair = sum N_i^2 / (B N_max^2): valid fraction of the padded pair envelope."""
    lengths = list(lengths)
    if not lengths or max(lengths) == 0:
        return 1.0
    return sum(n * n for n in lengths) / (len(lengths) * max(lengths) ** 2)
