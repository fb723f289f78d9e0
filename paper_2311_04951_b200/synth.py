"""Seeded synthetic inputs: architectures, weights, prompts, uniforms, draft rows.

This module only *draws data*.  It contains none of the arithmetic of the
method (no decoder math, no softmax, no acceptance test): both the CPU oracle's
tests and the CUDA path's tests feed on the arrays produced here, so that the
two sides see bit-identical inputs without sharing any computation.

Tensor order of a model (``tensor_names``):

    tok_emb [V,d], pos_emb [max_pos,d] (learned positions only, else None),
    per layer: ln1_g, ln1_b, w_qkv [3d,d], b_qkv, w_o [d,d], b_o,
               ln2_g, ln2_b, w_in [F or 2F,d], b_in, w_out [d,F], b_out,
    lnf_g, lnf_b, w_lm [V,d] (None when the LM head is tied to tok_emb)

Matrices are stored in the model dtype (fp32, or bf16 bit patterns as uint16);
vectors (gains, biases) are always fp32.  Absent tensors (RMSNorm has no bias,
bias-free families have no linear bias) are None.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np

NORM_LAYERNORM, NORM_RMS = 0, 1
ACT_GELU, ACT_SWIGLU = 0, 1
POS_LEARNED, POS_ROTARY = 0, 1
DT_F32, DT_BF16 = 0, 1

PER_LAYER = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
             "ln2_g", "ln2_b", "w_in", "b_in", "w_out", "b_out")


@dataclasses.dataclass(frozen=True)
class Arch:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    max_pos: int
    norm: int
    act: int
    pos: int
    parallel_residual: int
    has_bias: int
    tie_lm_head: int
    dtype: int
    rotary_dim: int
    rotary_base: float = 10000.0
    norm_eps: float = 1e-5

    def replace(self, **kw) -> "Arch":
        return dataclasses.replace(self, **kw)

    @property
    def d_in(self) -> int:
        """Rows of the MLP input projection (gate and up stacked for SwiGLU)."""
        return 2 * self.d_ff if self.act == ACT_SWIGLU else self.d_ff


def gpt2_like(L, d, H, F, V, max_pos, dtype=DT_F32) -> Arch:
    return Arch(L, d, H, d // H, F, V, max_pos, NORM_LAYERNORM, ACT_GELU, POS_LEARNED,
                0, 1, 1, dtype, 0)


def neox_like(L, d, H, F, V, dtype=DT_BF16) -> Arch:
    return Arch(L, d, H, d // H, F, V, 0, NORM_LAYERNORM, ACT_GELU, POS_ROTARY,
                1, 1, 0, dtype, d // H)


def llama_like(L, d, H, F, V, dtype=DT_BF16) -> Arch:
    return Arch(L, d, H, d // H, F, V, 0, NORM_RMS, ACT_SWIGLU, POS_ROTARY,
                0, 0, 0, dtype, d // H)


# The named workloads: (target, draft, draft_kind).  draft_kind "prefix:n" means the
# draft is the target's first n layers plus its final norm and LM head.
PRESETS: Dict[str, dict] = {
    "tiny": dict(target=gpt2_like(4, 256, 4, 1024, 1024, 256), draft="prefix:1",
                 batch=1, prompt=32, K=4, temperature=1.0, new_tokens=64,
                 seeds=dict(w=1, prompt=2, u=3)),
    "neox-1.4b": dict(target=neox_like(24, 2048, 16, 8192, 50304),
                      draft=neox_like(12, 768, 12, 3072, 50304),
                      batch=1, prompt=128, K=5, temperature=0.8, new_tokens=256,
                      seeds=dict(w=11, wd=12, prompt=13, u=14)),
    "neox-2.7b": dict(target=neox_like(32, 2560, 32, 10240, 50304), draft="prefix:4",
                      batch=1, prompt=512, K=8, temperature=0.0, new_tokens=512,
                      seeds=dict(w=21, prompt=23, u=24)),
    # the shape pair of the paper's own experiment (Section "Experimental results": a 12B target with a 3B draft,
    # K = 5, 40 and 100 new tokens): NeoX-style blocks, 36 layers x 5120 (40 heads of 128, rotary on a quarter of
    # the head) and 32 layers x 2560 (32 heads of 80); random-init stand-ins, batch 1
    "neox-12b": dict(target=neox_like(36, 5120, 40, 20480, 50304).replace(rotary_dim=32),
                     draft=neox_like(32, 2560, 32, 10240, 50304),
                     batch=1, prompt=128, K=5, temperature=1.0, new_tokens=100,
                     seeds=dict(w=41, wd=42, prompt=43, u=44)),
    "llama-7b": dict(target=llama_like(32, 4096, 32, 11008, 32000),
                     draft=llama_like(4, 1024, 16, 2752, 32000),
                     batch=8, prompt=2048, K=4, temperature=1.0, new_tokens=256,
                     seeds=dict(w=31, wd=32, prompt=33, u=34)),
}


def tensor_names(arch: Arch) -> List[str]:
    names = ["tok_emb", "pos_emb"]
    for l in range(arch.n_layers):
        names += [f"l{l}.{n}" for n in PER_LAYER]
    names += ["lnf_g", "lnf_b", "w_lm"]
    return names


def tensor_shape(arch: Arch, name: str) -> Optional[tuple]:
    """Shape of a tensor, or None when the architecture does not have it."""
    d, F, V = arch.d_model, arch.d_ff, arch.vocab
    base = name.split(".")[-1]
    ln_bias = arch.norm == NORM_LAYERNORM
    table = {
        "tok_emb": (V, d),
        "pos_emb": (arch.max_pos, d) if arch.pos == POS_LEARNED else None,
        "ln1_g": (d,), "ln1_b": (d,) if ln_bias else None,
        "w_qkv": (3 * d, d), "b_qkv": (3 * d,) if arch.has_bias else None,
        "w_o": (d, d), "b_o": (d,) if arch.has_bias else None,
        "ln2_g": (d,), "ln2_b": (d,) if ln_bias else None,
        "w_in": (arch.d_in, d), "b_in": (arch.d_in,) if arch.has_bias else None,
        "w_out": (d, F), "b_out": (d,) if arch.has_bias else None,
        "lnf_g": (d,), "lnf_b": (d,) if ln_bias else None,
        "w_lm": None if arch.tie_lm_head else (V, d),
    }
    return table[base]


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal(rng: np.random.Generator, shape, std: float, mean: float = 0.0) -> np.ndarray:
    out = rng.standard_normal(shape, dtype=np.float32)
    out *= np.float32(std)
    if mean:
        out += np.float32(mean)
    return out


def gen_tensor(arch: Arch, seed: int, index: int, name: str,
               late_scale: float = 1.0, late_from: int = 0) -> Optional[np.ndarray]:
    """One tensor of a model, drawn from its own stream (seed, index).

    Every matrix, bias and embedding ~ N(0, 0.02); norm gains ~ 1 + N(0, 0.02).
    ``late_scale`` multiplies the output projections (w_o, w_out, b_o, b_out) of
    layers >= ``late_from`` so that an early-exit draft stays correlated with the
    full model.
    """
    shape = tensor_shape(arch, name)
    if shape is None:
        return None
    rng = np.random.Generator(np.random.Philox(key=[seed, index]))
    base = name.split(".")[-1]
    if base.endswith("_g"):
        return _normal(rng, shape, 0.02, 1.0)
    t = _normal(rng, shape, 0.02)
    if "." in name and base in ("w_o", "w_out", "b_o", "b_out"):
        layer = int(name.split(".")[0][1:])
        if layer >= late_from and late_scale != 1.0:
            t *= np.float32(late_scale)
    if len(shape) == 2 and arch.dtype == DT_BF16:
        return f32_to_bf16_bits(t)
    return t


def gen_weights(arch: Arch, seed: int, late_scale: float = 1.0,
                late_from: int = 0) -> List[Optional[np.ndarray]]:
    return [gen_tensor(arch, seed, i, n, late_scale, late_from)
            for i, n in enumerate(tensor_names(arch))]


def prefix_draft(arch: Arch, weights: List, n_layers: int):
    """Early-exit draft: the first n layers + final norm + LM head of a model (shared arrays)."""
    d_arch = arch.replace(n_layers=n_layers)
    keep = 2 + len(PER_LAYER) * n_layers
    return d_arch, list(weights[:keep]) + list(weights[-3:])


def gen_prompt(seed: int, batch: int, length: int, vocab: int) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=[seed, 0]))
    return rng.integers(0, vocab, size=(batch, length), dtype=np.int32)


def gen_uniforms(seed: int, seq: int, iteration: int, count: int) -> np.ndarray:
    """`count` uniforms in [0,1) on the 24-bit grid k*2^-24, keyed by (seed, seq, iteration)."""
    rng = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ seq, iteration]))
    k = rng.integers(0, 1 << 24, size=count, dtype=np.uint32)
    return (k.astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)


def gen_dirichlet_rows(seed: int, rows: int, vocab: int, alpha: float = 0.1) -> np.ndarray:
    """Rows ~ Dirichlet(alpha) over the vocabulary (gamma draws in float64, normalised, cast to
    fp32; exact zeros can occur)."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 1]))
    g = rng.standard_gamma(alpha, size=(rows, vocab))
    g /= g.sum(axis=1, keepdims=True)
    return g.astype(np.float32)


def draw_tokens_from_rows(seed: int, rows: np.ndarray) -> np.ndarray:
    """One token per row, distributed as the row (used to make draft tokens for supplied q)."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 2]))
    out = np.empty(rows.shape[0], dtype=np.int32)
    for i, r in enumerate(rows):
        out[i] = rng.choice(r.shape[0], p=r.astype(np.float64) / r.astype(np.float64).sum())
    return out


def gen_logits(seed: int, rows: int, vocab: int, std: float = 1.0) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=[seed, 3]))
    return _normal(rng, (rows, vocab), std)


def gen_kv_fill(seed: int, shape, dtype: int) -> np.ndarray:
    """Seeded N(0,1) cache contents (bf16 bit patterns or fp32)."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 4]))
    t = rng.standard_normal(shape, dtype=np.float32)
    return f32_to_bf16_bits(t) if dtype == DT_BF16 else t
