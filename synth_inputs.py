"""Seeded synthetic input generators shared by the tests, the benchmark and the smoke check.

This module only draws random tensors of the shapes and distributions the workloads call
for. It contains none of the quantization or inner-product arithmetic: it never rounds a
weight onto a lattice, never builds an exchange, never forms a dot product. Both the CPU
oracle's tests and the CUDA path's tests take their inputs from here so that the two sides
see the same bytes without sharing any of the method's code.

Workload shapes (LLaMA-2-7B / 70B and ViT-B/16 linears) are used as shapes only; all values
are synthetic.
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------------------
# Shapes (N_out, K_in) of the linears the workloads name.
# ----------------------------------------------------------------------------------------
LLAMA2_7B_LINEARS = (
    ("q_proj", 4096, 4096),
    ("k_proj", 4096, 4096),
    ("v_proj", 4096, 4096),
    ("o_proj", 4096, 4096),
    ("gate_proj", 11008, 4096),
    ("up_proj", 11008, 4096),
    ("down_proj", 4096, 11008),
)
LLAMA2_7B_LAYERS = 32

LLAMA2_70B_LINEARS = (
    ("attn_qo", 8192, 8192),
    ("mlp_gate_up", 28672, 8192),
    ("mlp_down", 8192, 28672),
    ("gqa_kv", 1024, 8192),
)

VIT_B16_LINEARS = (
    ("qkv", 2304, 768),
    ("attn_out", 768, 768),
    ("mlp_fc1", 3072, 768),
    ("mlp_fc2", 768, 3072),
)
VIT_B16_TOKENS = 197 * 64


def _rng(seed: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence(int(seed)))


# ----------------------------------------------------------------------------------------
# Weights
# ----------------------------------------------------------------------------------------
def gaussian_weights(n_out: int, k_in: int, std: float = 0.02, seed: int = 0) -> np.ndarray:
    """fp32 [n_out][k_in] ~ N(0, std^2)."""
    return (_rng(seed).standard_normal((n_out, k_in)) * std).astype(np.float32)


def weights_with_outlier_channels(n_out: int, k_in: int, std: float = 0.02, frac: float = 0.01,
                                  scale: float = 20.0, seed: int = 0) -> np.ndarray:
    """N(0, std^2) weights with a seeded `frac` of the input channels multiplied by `scale`."""
    rng = _rng(seed)
    w = rng.standard_normal((n_out, k_in)) * std
    n_outl = max(1, int(round(frac * k_in)))
    cols = rng.choice(k_in, size=n_outl, replace=False)
    w[:, cols] *= scale
    return w.astype(np.float32)


def weights_with_student_t_channels(n_out: int, k_in: int, std: float = 0.015, frac: float = 0.01,
                                    nu: float = 4.0, scale: float = 10.0, seed: int = 0) -> np.ndarray:
    """N(0, std^2) weights; a seeded `frac` of input channels redrawn as std*scale*t_nu."""
    rng = _rng(seed)
    w = rng.standard_normal((n_out, k_in)) * std
    n_outl = max(1, int(round(frac * k_in)))
    cols = rng.choice(k_in, size=n_outl, replace=False)
    w[:, cols] = rng.standard_t(nu, size=(n_out, n_outl)) * (std * scale)
    return w.astype(np.float32)


# ----------------------------------------------------------------------------------------
# Activations
# ----------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = (u + 0x7FFF + lsb) >> 16
    return r.astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    u = (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16)
    return u.view(np.float32).astype(np.float64)


def bf16_activations(m: int, k_in: int, seed: int = 0, std: float = 1.0) -> np.ndarray:
    """[m][k_in] activations ~ N(0, std^2) rounded to bf16; returned as uint16 bit patterns."""
    x = (_rng(seed).standard_normal((m, k_in)) * std).astype(np.float32)
    return f32_to_bf16_bits(x)


def f32_activations(m: int, k_in: int, seed: int = 0, std: float = 1.0) -> np.ndarray:
    """fp32 [m][k_in] ~ N(0, std^2), the source of the int8 activation path."""
    return (_rng(seed).standard_normal((m, k_in)) * std).astype(np.float32)


def int8_activations(m: int, k_in: int, seed: int = 0):
    """Uniform int8 activations in [-127, 127] plus positive per-token fp32 scales."""
    rng = _rng(seed)
    xq = rng.integers(-127, 128, size=(m, k_in), dtype=np.int16).astype(np.int8)
    sx = rng.uniform(0.005, 0.05, size=(m,)).astype(np.float32)
    return xq, sx


# ----------------------------------------------------------------------------------------
# Random quantized records (valid code / metadata / coefficient fields drawn directly),
# used where a shape is too large to run the CPU quantizer over in a test or benchmark.
# ----------------------------------------------------------------------------------------
def random_quantized(n_out: int, k_in: int, group: int, wbits: int, seed: int = 0,
                     coef_std: float = 0.05):
    """Draw per-weight codes in [0, 2^wbits), per-8-weight 6-bit records and fp16 coefficient
    pairs. Code frequencies follow a fixed table that puts more mass on the small-magnitude
    states, as a Gaussian block normalised by its largest entry does.

    Returns (codes u8 [N][K], meta u8 [N][K/8], coef fp16 [N][K/group][2]).
    """
    assert k_in % group == 0 and group % 8 == 0
    rng = _rng(seed)
    n_codes = 1 << wbits
    half = n_codes // 2
    # weight of exponent index e (0 = largest magnitude) grows with e
    w_e = np.array([1.0 + 1.5 * e for e in range(half)])
    p = np.concatenate([w_e, w_e])
    p = p / p.sum()
    codes = rng.choice(n_codes, size=(n_out, k_in), p=p).astype(np.uint8)
    meta = rng.integers(0, 64, size=(n_out, k_in // 8), dtype=np.uint8)
    c = rng.standard_normal((n_out, k_in // group, 2)) * coef_std
    c[..., 0] = np.abs(c[..., 0]) + 0.25 * coef_std
    c[..., 1] = np.abs(c[..., 1]) * 0.3
    coef = c.astype(np.float16)
    return codes, meta, coef


def random_int8_coefficients(n_out: int, n_groups: int, seed: int = 0):
    """Integer coefficient pairs in [-127, 127] and positive per-output-channel scales."""
    rng = _rng(seed)
    cq = rng.integers(-127, 128, size=(n_out, n_groups, 2), dtype=np.int16).astype(np.int8)
    sc = rng.uniform(1e-4, 1e-3, size=(n_out, 2)).astype(np.float32)
    return cq, sc


def sample_rows(n_out: int, count: int, seed: int = 0) -> np.ndarray:
    """Seeded sorted sample of output rows, always including the first and last row."""
    count = min(count, n_out)
    rng = _rng(seed)
    rows = set(rng.choice(n_out, size=count, replace=False).tolist())
    rows.update((0, n_out - 1))
    return np.array(sorted(rows), dtype=np.int64)
