"""Model-shaped tensor lists and seeded synthetic inputs.

This module holds no optimizer arithmetic.  It describes the parameter tensors
of the benchmark workloads (shape, partition kind, gradient dtype) and draws
their parameters and per-step gradients from seeded generators, on whatever
device the caller names.  Both the CUDA library's callers and the CPU checker
used by the tests take their inputs from here, so they always see the same
bits.

Shapes follow the usual [out_features, in_features] row-major convention, so a
token row, an output neuron and an attention head are contiguous runs
(Algorithm 3 of the paper partitions along dim 0).

Gradient recipe: g = sigma_row * z with z ~ N(0, 1) fresh at every step and
sigma_row fixed per output row over the steps (1-D tensors: one sigma), cast
to the tensor's gradient dtype with round-to-nearest-even.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import torch

# Partition kinds and dtype codes (values of the library's C enums).
WHOLE, ROWS, HEADS, TOKENS, FIXED, PART = 0, 1, 2, 3, 4, 5
F32, BF16 = 0, 1

BASE_SEED = 20240616
_MASK = (1 << 64) - 1
_CHUNK = 1 << 25  # elements drawn per call, bounds temporary memory


@dataclass(frozen=True)
class TensorSpec:
    name: str
    rows: int
    cols: int
    kind: int
    n_heads: int = 0
    fixed_block_len: int = 0
    grad_dtype: int = F32
    apply_weight_decay: int = 1
    zipf_rows: bool = False      # embedding/output rows with Zipf-distributed magnitudes

    @property
    def numel(self) -> int:
        return self.rows * self.cols

    @property
    def block_len(self) -> int:
        if self.kind in (WHOLE, PART):      # PART: the local part of a longer block is the tensor's one block
            return self.numel
        if self.kind in (ROWS, TOKENS):
            return self.cols
        if self.kind == HEADS:
            return (self.rows // self.n_heads) * self.cols
        return self.fixed_block_len

    @property
    def n_blocks(self) -> int:
        return self.numel // self.block_len


@dataclass(frozen=True)
class GradRecipe:
    log10_lo: float = -4.0
    log10_hi: float = -1.0
    outlier_prob: float = 0.0     # Bernoulli mask over rows, fixed over steps
    outlier_scale: float = 1.0
    zipf_exponent: float = 1.1
    zipf_scale: float = 0.1
    chunk: int = 0                # >0: one sigma per `chunk` consecutive elements (flat tensors)


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    tensors: List[TensorSpec]
    recipe: GradRecipe
    steps: int
    hparams: Dict[str, float] = field(default_factory=lambda: dict(
        lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1))

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)

    @property
    def n_blocks(self) -> int:
        return sum(t.n_blocks for t in self.tensors)


# ----------------------------------------------------------------------------
# model shapes
# ----------------------------------------------------------------------------

def gpt2_like(n_layers: int, d_model: int, n_heads: int, d_ff: int, vocab: int, *,
              grad_dtype: int, tied: bool, pos_rows: int = 0, linear_bias: bool = False,
              norm_bias: bool = True) -> List[TensorSpec]:
    """GPT-2-style decoder: separate q/k/v weights (a fused qkv tensor is three
    descriptors), LayerNorm weights (+biases), optional linear biases."""
    t: List[TensorSpec] = []
    gd = dict(grad_dtype=grad_dtype)

    def whole(name: str, n: int) -> None:
        t.append(TensorSpec(name, 1, n, WHOLE, **gd))

    t.append(TensorSpec("embed.wte", vocab, d_model, TOKENS, **gd))
    if pos_rows:
        t.append(TensorSpec("embed.wpe", pos_rows, d_model, TOKENS, **gd))
    for i in range(n_layers):
        pre = f"h.{i}."
        whole(pre + "ln_1.weight", d_model)
        if norm_bias:
            whole(pre + "ln_1.bias", d_model)
        t.append(TensorSpec(pre + "attn.query.weight", d_model, d_model, HEADS, n_heads=n_heads, **gd))
        t.append(TensorSpec(pre + "attn.key.weight", d_model, d_model, HEADS, n_heads=n_heads, **gd))
        t.append(TensorSpec(pre + "attn.value.weight", d_model, d_model, ROWS, **gd))
        if linear_bias:
            whole(pre + "attn.query.bias", d_model)
            whole(pre + "attn.key.bias", d_model)
            whole(pre + "attn.value.bias", d_model)
        t.append(TensorSpec(pre + "attn.proj.weight", d_model, d_model, ROWS, **gd))
        if linear_bias:
            whole(pre + "attn.proj.bias", d_model)
        whole(pre + "ln_2.weight", d_model)
        if norm_bias:
            whole(pre + "ln_2.bias", d_model)
        t.append(TensorSpec(pre + "mlp.fc.weight", d_ff, d_model, ROWS, **gd))
        if linear_bias:
            whole(pre + "mlp.fc.bias", d_ff)
        t.append(TensorSpec(pre + "mlp.proj.weight", d_model, d_ff, ROWS, **gd))
        if linear_bias:
            whole(pre + "mlp.proj.bias", d_model)
    whole("ln_f.weight", d_model)
    if norm_bias:
        whole("ln_f.bias", d_model)
    if not tied:
        t.append(TensorSpec("output.weight", vocab, d_model, TOKENS, **gd))
    return t


def llama_like(n_layers: int, d_model: int, n_heads: int, n_kv_heads: int, d_ff: int, vocab: int, *,
               grad_dtype: int = BF16, zipf_vocab: bool = False) -> List[TensorSpec]:
    """Llama-style decoder: RMSNorm weights, SwiGLU MLP, optional grouped KV heads."""
    head_dim = d_model // n_heads
    kv_rows = n_kv_heads * head_dim
    gd = dict(grad_dtype=grad_dtype)
    t: List[TensorSpec] = [TensorSpec("embed_tokens.weight", vocab, d_model, TOKENS, zipf_rows=zipf_vocab, **gd)]
    for i in range(n_layers):
        pre = f"layers.{i}."
        t.append(TensorSpec(pre + "attention_norm.weight", 1, d_model, WHOLE, **gd))
        t.append(TensorSpec(pre + "attention.query.weight", d_model, d_model, HEADS, n_heads=n_heads, **gd))
        t.append(TensorSpec(pre + "attention.key.weight", kv_rows, d_model, HEADS, n_heads=n_kv_heads, **gd))
        t.append(TensorSpec(pre + "attention.value.weight", kv_rows, d_model, ROWS, **gd))
        t.append(TensorSpec(pre + "attn.proj.weight", d_model, d_model, ROWS, **gd))
        t.append(TensorSpec(pre + "ffn_norm.weight", 1, d_model, WHOLE, **gd))
        t.append(TensorSpec(pre + "mlp.gate.weight", d_ff, d_model, ROWS, **gd))
        t.append(TensorSpec(pre + "mlp.up.weight", d_ff, d_model, ROWS, **gd))
        t.append(TensorSpec(pre + "mlp.down.weight", d_model, d_ff, ROWS, **gd))
    t.append(TensorSpec("norm.weight", 1, d_model, WHOLE, **gd))
    t.append(TensorSpec("output.weight", vocab, d_model, TOKENS, zipf_rows=zipf_vocab, **gd))
    return t


def flat_tensor(numel: int, block_len: int, grad_dtype: int = F32) -> List[TensorSpec]:
    return [TensorSpec("flat", 1, numel, FIXED, fixed_block_len=block_len, grad_dtype=grad_dtype)]


def tiny_gpt2() -> Workload:
    """2 layers, d_model 128, 4 heads, d_ff 512, vocab 1024, untied, fp32 gradients."""
    return Workload("tiny-gpt2", 1,
                    gpt2_like(2, 128, 4, 512, 1024, grad_dtype=F32, tied=False),
                    GradRecipe(-4.0, -1.0), steps=10)


def gpt2_small(n_layers: int = 12) -> Workload:
    """GPT-2-small shapes (124M): tied embedding, 1024x768 positions, linear biases."""
    return Workload("gpt2-small", 2,
                    gpt2_like(n_layers, 768, 12, 3072, 50304, grad_dtype=BF16, tied=True,
                              pos_rows=1024, linear_bias=True),
                    GradRecipe(-5.0, -1.0), steps=100)


def llama2_7b(n_layers: int = 32, vocab: int = 32000) -> Workload:
    """Llama-2-7B shapes; 1% of rows carry gradients 100x larger (outliers)."""
    return Workload("llama2-7b", 3,
                    llama_like(n_layers, 4096, 32, 32, 11008, vocab),
                    GradRecipe(-5.0, -1.0, outlier_prob=0.01, outlier_scale=100.0), steps=20)


def llama3_8b(n_layers: int = 32, vocab: int = 128256) -> Workload:
    """Llama-3-8B shapes with 8 KV heads; Zipf(1.1) row magnitudes on embed/output."""
    return Workload("llama3-8b", 4,
                    llama_like(n_layers, 4096, 32, 8, 14336, vocab, zipf_vocab=True),
                    GradRecipe(-5.0, -1.0), steps=20)


def flat_sweep(block_len: int, numel: int = 1 << 30) -> Workload:
    """One flat fp32 tensor, blocks of `block_len`, sigma per 64-element chunk."""
    return Workload(f"flat-L{block_len}", 5, flat_tensor(numel, block_len),
                    GradRecipe(-4.0, 0.0, chunk=64), steps=10)


def scaled_rows(w: Workload, max_rows: int, name: Optional[str] = None) -> Workload:
    """Same tensors with every 2-D tensor cut to at most `max_rows` rows (heads
    kept whole), preserving every block length of the full workload.  Used for
    parity cases the CPU checker can finish in seconds."""
    out = []
    for t in w.tensors:
        if t.rows <= max_rows or t.kind == WHOLE:
            out.append(t)
        elif t.kind == HEADS:
            hd = t.rows // t.n_heads
            nh = max(1, max_rows // hd)
            out.append(replace(t, rows=nh * hd, n_heads=nh))
        else:
            out.append(replace(t, rows=max_rows))
    return replace(w, name=name or (w.name + f"-rows{max_rows}"), tensors=out)


# ----------------------------------------------------------------------------
# seeded generators
# ----------------------------------------------------------------------------

def mix_seed(*parts: int) -> int:
    """Deterministic 63-bit seed from integers (splitmix64 finaliser chain)."""
    x = 0x9E3779B97F4A7C15
    for p in parts:
        x = (x ^ (int(p) & _MASK)) & _MASK
        x = (x + 0x9E3779B97F4A7C15) & _MASK
        x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
        x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _MASK
        x = x ^ (x >> 31)
    return x & ((1 << 63) - 1)


def _gen(device, *parts: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(mix_seed(BASE_SEED, *parts))
    return g


def torch_dtype(code: int) -> torch.dtype:
    return torch.bfloat16 if code == BF16 else torch.float32


def gen_param(w: Workload, index: int, device="cpu") -> torch.Tensor:
    """fp32 N(0, 0.02^2) parameters of tensor `index`, flat."""
    t = w.tensors[index]
    out = torch.empty(t.numel, dtype=torch.float32, device=device)
    g = _gen(device, w.config_id, 0, index, 1)
    for lo in range(0, t.numel, _CHUNK):
        out[lo:lo + _CHUNK].normal_(0.0, 0.02, generator=g)
    return out


def row_sigmas(w: Workload, index: int, device="cpu") -> torch.Tensor:
    """Per-row (or per-chunk) gradient scale of tensor `index`; fixed over steps."""
    t, r = w.tensors[index], w.recipe
    n = t.numel // r.chunk if r.chunk else t.rows
    g = _gen(device, w.config_id, 0, index, 2)
    if t.zipf_rows:
        perm = torch.randperm(n, generator=g, device=device)
        return (r.zipf_scale * (perm.to(torch.float64) + 1.0).pow(-r.zipf_exponent)).to(torch.float32)
    u = torch.rand(n, generator=g, device=device, dtype=torch.float32)
    sig = torch.pow(10.0, r.log10_lo + (r.log10_hi - r.log10_lo) * u)
    if r.outlier_prob > 0.0:
        mask = torch.rand(n, generator=g, device=device, dtype=torch.float32) < r.outlier_prob
        sig = torch.where(mask, sig * r.outlier_scale, sig)
    return sig


def gen_grad(w: Workload, index: int, step: int, device="cpu",
             out: Optional[torch.Tensor] = None, sigmas: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Gradient of tensor `index` at `step` (1-based), flat, in its gradient dtype."""
    t, r = w.tensors[index], w.recipe
    if out is None:
        out = torch.empty(t.numel, dtype=torch_dtype(t.grad_dtype), device=device)
    if sigmas is None:
        sigmas = row_sigmas(w, index, device)
    width = r.chunk if r.chunk else t.cols
    g = _gen(device, w.config_id, step, index, 3)
    rows_per = max(1, _CHUNK // width)
    n_rows = t.numel // width
    out2 = out.view(n_rows, width)
    for lo in range(0, n_rows, rows_per):
        hi = min(n_rows, lo + rows_per)
        z = torch.randn(hi - lo, width, generator=g, device=device, dtype=torch.float32)
        z.mul_(sigmas[lo:hi].unsqueeze(1))
        out2[lo:hi].copy_(z)          # RNE cast when the gradient dtype is bf16
    return out


def algorithmic_bytes_per_param(t: TensorSpec, onchip_limit: int) -> float:
    """Bytes the update must move per parameter of tensor `t`: g once (twice if
    one block exceeds `onchip_limit` elements), m and p read and written, v
    read and written once per block."""
    gsz = 2 if t.grad_dtype == BF16 else 4
    g_reads = 2 if t.block_len > onchip_limit else 1
    return g_reads * gsz + 16 + 8.0 / t.block_len


def log2_int(n: int) -> int:
    return int(math.log2(n))
