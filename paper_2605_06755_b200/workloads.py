"""Seeded synthetic inputs and tensor-list shapes.

This module holds NONE of the method's arithmetic: it only draws random numbers
and lists tensor shapes, so that the CUDA path, the CPU oracle and the benchmark
can all be fed the same bits.  The real gradients of the paper come from RL
training runs; these are stand-ins with the sizes, dtypes and rough magnitudes
of that workload.

Recipe for the LLM-shaped cases ("N(0, x)" means standard deviation x):
  theta ~ N(0, 0.02) fp32;   g0f ~ N(0, 1e-3) fp32;
  g0 = bf16(g0f),  g1 = bf16(g0f + N(0, 1e-4)),  g_slow = bf16(g0f + N(0, 2e-4)),
  round-to-nearest-even; optionally a fraction of g0 is zeroed so that the
  inactive branch is taken at a realistic rate.
Recipe for the diagonal-quadratic surrogate f = sum(a x^2 / 2 - b x):
  a ~ U[0.1, 1), b ~ N(0, 1), theta0 ~ N(0, 1), fp32.
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np


# ----------------------------------------------------------------------------
# tensor-list shapes
# ----------------------------------------------------------------------------
def decoder_shapes(layers: int, hidden: int, ffn: int, q_heads: int, kv_heads: int,
                   head_dim: int, vocab: int, qkv_bias: bool) -> List[Tuple[str, int]]:
    """(name, numel) of every parameter tensor of a Llama/Qwen-style decoder with
    an untied embedding and LM head and RMSNorm vectors."""
    out: List[Tuple[str, int]] = [("embed_tokens", vocab * hidden)]
    q_out = q_heads * head_dim
    kv_out = kv_heads * head_dim
    for l in range(layers):
        p = f"layers.{l}."
        out.append((p + "input_layernorm", hidden))
        out.append((p + "q_proj.weight", q_out * hidden))
        if qkv_bias:
            out.append((p + "q_proj.bias", q_out))
        out.append((p + "k_proj.weight", kv_out * hidden))
        if qkv_bias:
            out.append((p + "k_proj.bias", kv_out))
        out.append((p + "v_proj.weight", kv_out * hidden))
        if qkv_bias:
            out.append((p + "v_proj.bias", kv_out))
        out.append((p + "o_proj.weight", hidden * q_out))
        out.append((p + "post_attention_layernorm", hidden))
        out.append((p + "gate_proj.weight", ffn * hidden))
        out.append((p + "up_proj.weight", ffn * hidden))
        out.append((p + "down_proj.weight", hidden * ffn))
    out.append(("norm", hidden))
    out.append(("lm_head", vocab * hidden))
    return out


def qwen25_7b_shapes(layers: int = 28) -> List[Tuple[str, int]]:
    """Qwen2.5-7B-shaped list: hidden 3584, FFN 18944, 28 q / 4 kv heads of dim 128,
    vocab 152064, q/k/v biases.  28 layers -> 7,615,616,512 parameters in 339 tensors."""
    return decoder_shapes(layers, 3584, 18944, 28, 4, 128, 152064, qkv_bias=True)


def llama31_8b_shapes(layers: int = 32) -> List[Tuple[str, int]]:
    """Llama-3.1-8B-shaped list: hidden 4096, FFN 14336, 32 q / 8 kv heads of dim 128,
    vocab 128256.  32 layers -> 8,030,261,248 parameters in 291 tensors."""
    return decoder_shapes(layers, 4096, 14336, 32, 8, 128, 128256, qkv_bias=False)


def lora_qwen25_7b_shapes(rank: int = 128, layers: int = 28) -> List[Tuple[str, int]]:
    """Rank-`rank` LoRA adapters on the q, k, v, o projections of a Qwen2.5-7B-shaped
    decoder (the paper's 7B setting): per layer four A matrices [rank x in] and four B
    matrices [out x rank].  rank 128 -> 224 tensors of 65,536 or 458,752 elements,
    80,740,352 parameters."""
    hidden, q_out, kv_out = 3584, 28 * 128, 4 * 128
    out: List[Tuple[str, int]] = []
    for l in range(layers):
        for name, fan_in, fan_out in (("q_proj", hidden, q_out), ("k_proj", hidden, kv_out),
                                      ("v_proj", hidden, kv_out), ("o_proj", q_out, hidden)):
            out.append((f"layers.{l}.{name}.lora_A", rank * fan_in))
            out.append((f"layers.{l}.{name}.lora_B", fan_out * rank))
    return out


FLAT_QWEN25_1P5B = 1_540_000_000   # "flat 1.54e9-param buffer"


def scaled_shapes(shapes: List[Tuple[str, int]], max_numel: int) -> List[Tuple[str, int]]:
    """The same list with every tensor capped at max_numel elements (sizes kept
    odd-shaped: the cap is applied to numel, small tensors stay as they are)."""
    return [(name, min(n, max_numel)) for name, n in shapes]


# ----------------------------------------------------------------------------
# diagonal-quadratic surrogate (numpy; sizes up to ~1e8)
# ----------------------------------------------------------------------------
def quadratic_surrogate(n: int, seed: int = 0):
    """a, b, theta0 as float32 numpy arrays."""
    rng = np.random.default_rng(seed)
    a = rng.uniform(0.1, 1.0, size=n).astype(np.float32)
    b = rng.standard_normal(n, dtype=np.float32)
    theta0 = rng.standard_normal(n, dtype=np.float32)
    return a, b, theta0


# ----------------------------------------------------------------------------
# LLM-shaped gradients (numpy for small cases, torch on the device for large)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16).
    A data-format conversion; NaN payloads are kept quiet."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    is_nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    rounded = np.where(is_nan, (u >> np.uint32(16)) | np.uint32(0x0040), rounded)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def llm_inputs_numpy(n: int, seed: int, grad_dtype: str = "bf16", zero_frac: float = 0.0,
                     warm_state: bool = False):
    """theta, m, v (fp32) and g0, g1, g_slow for a flat vector of n parameters.
    Gradients come back as uint16 bfloat16 bit patterns (grad_dtype='bf16') or
    float32 arrays ('f32')."""
    rng = np.random.default_rng(seed)
    theta = (0.02 * rng.standard_normal(n, dtype=np.float32)).astype(np.float32)
    g0f = (1e-3 * rng.standard_normal(n, dtype=np.float32)).astype(np.float32)
    g1f = g0f + (1e-4 * rng.standard_normal(n, dtype=np.float32)).astype(np.float32)
    gsf = g0f + (2e-4 * rng.standard_normal(n, dtype=np.float32)).astype(np.float32)
    if zero_frac > 0.0:
        g0f = np.where(rng.random(n) < zero_frac, np.float32(0), g0f).astype(np.float32)
    if warm_state:
        m = (1e-3 * rng.standard_normal(n, dtype=np.float32)).astype(np.float32)
        v = (1e-6 * rng.random(n, dtype=np.float32)).astype(np.float32)
    else:
        m = np.zeros(n, dtype=np.float32)
        v = np.zeros(n, dtype=np.float32)
    if grad_dtype == "bf16":
        return theta, m, v, f32_to_bf16_bits(g0f), f32_to_bf16_bits(g1f), f32_to_bf16_bits(gsf)
    return theta, m, v, g0f, g1f.astype(np.float32), gsf.astype(np.float32)


def fill_llm_inputs_torch(theta, m, v, g0, g1, g_slow, seed: int, zero_frac: float = 0.0,
                          block: int = 1 << 26):
    """Fill flat device tensors in place, in bounded blocks (torch ops only; used
    for sizes that numpy on the host would take minutes to draw).  theta/m/v are
    fp32; g0/g1/g_slow are bf16 or fp32 tensors of the same length; g_slow may be
    None.  m and v are zeroed."""
    import torch

    gen = torch.Generator(device=theta.device)
    gen.manual_seed(seed)
    n = theta.numel()
    m.zero_()
    v.zero_()
    for s in range(0, n, block):
        e = min(n, s + block)
        k = e - s
        theta[s:e] = torch.randn(k, generator=gen, device=theta.device, dtype=torch.float32) * 0.02
        g0f = torch.randn(k, generator=gen, device=theta.device, dtype=torch.float32) * 1e-3
        g1[s:e] = (g0f + torch.randn(k, generator=gen, device=theta.device,
                                     dtype=torch.float32) * 1e-4).to(g1.dtype)
        if g_slow is not None:
            g_slow[s:e] = (g0f + torch.randn(k, generator=gen, device=theta.device,
                                             dtype=torch.float32) * 2e-4).to(g_slow.dtype)
        if zero_frac > 0.0:
            mask = torch.rand(k, generator=gen, device=theta.device) < zero_frac
            g0f = torch.where(mask, torch.zeros_like(g0f), g0f)
        g0[s:e] = g0f.to(g0.dtype)
        del g0f
