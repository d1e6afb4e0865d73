"""Seeded synthetic workloads: parameter-shape lists and gradient generators.

This module holds none of the optimizer's arithmetic. It only names tensor shapes (the public
architecture dimensions of the models the paper trains) and draws seeded random parameters and
gradients; the CUDA path and the CPU oracle are both fed from the same materialised buffers.

Gradient recipe (imitates the fixed-row / fixed-column outlier structure of Sec. 3, Fig. 2):
for a rows x cols tensor draw once a_i = exp(N(0,1)), b_j = exp(N(0,1)) and an outlier mask with
probability `outlier_p` (positions fixed across steps); each step draw z_ij ~ N(0,1) and set
g_ij = z_ij * a_i * b_j * (100 on the mask, else 1). One-dimensional tensors use a_i only.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

BASE_SEED = 20230901


@dataclass(frozen=True)
class TensorSpec:
    name: str
    rows: int
    cols: int
    ndim: int                # 1 or 2 (ndim 1: rows = numel, cols = 1); with `dims`: their number
    init: str = "normal"     # "normal" N(0, 0.02^2), "ones", "zeros"
    force_quant: bool = False
    sparse_rows: float = 0.0  # fraction of gradient rows zeroed each step (token-sparse embeddings)
    dims: tuple | None = None  # three or more axes (e.g. a convolution weight): rows = product of the leading extents

    @property
    def numel(self) -> int:
        return self.rows * self.cols

    @property
    def shape(self):
        if self.dims is not None:
            return tuple(self.dims)
        return (self.rows,) if self.ndim == 1 else (self.rows, self.cols)


@dataclass(frozen=True)
class Workload:
    name: str
    index: int               # position in the benchmark's list of configurations
    tensors: tuple
    lr: float
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.01
    grad_dtype: str = "f32"  # "f32" or "bf16"
    steps: int = 10

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)


def _mat(name, r, c, **kw):
    return TensorSpec(name, r, c, 2, **kw)


def _vec(name, n, init="zeros", **kw):
    return TensorSpec(name, n, 1, 1, init=init, **kw)


def single_matrix() -> Workload:
    """One 1024x4096 weight and its 4096-element bias (bias forced onto the quantized 1-D path)."""
    ts = (_mat("weight", 1024, 4096), _vec("bias", 4096, force_quant=True))
    return Workload("single_matrix_1024x4096", 0, ts, lr=1e-3, steps=10)


def transformer_base() -> Workload:
    """Encoder-decoder Transformer-base shapes: 6+6 layers, d_model 512, FFN 2048, vocab 32000."""
    d, ff, vocab = 512, 2048, 32000
    ts = [_mat("shared_embedding", vocab, d)]

    def attn(p):
        return [_mat(p + ".qkv.w", 3 * d, d), _vec(p + ".qkv.b", 3 * d),
                _mat(p + ".out.w", d, d), _vec(p + ".out.b", d)]

    def ffn(p):
        return [_mat(p + ".fc1.w", ff, d), _vec(p + ".fc1.b", ff),
                _mat(p + ".fc2.w", d, ff), _vec(p + ".fc2.b", d)]

    def ln(p):
        return [_vec(p + ".w", d, init="ones"), _vec(p + ".b", d)]

    for i in range(6):
        p = f"enc{i}"
        ts += attn(p + ".self") + ffn(p) + ln(p + ".ln1") + ln(p + ".ln2")
    for i in range(6):
        p = f"dec{i}"
        ts += attn(p + ".self") + attn(p + ".cross") + ffn(p) + ln(p + ".ln1") + ln(p + ".ln2") + ln(p + ".ln3")
    return Workload("transformer_base", 1, tuple(ts), lr=1e-3, steps=100)


def roberta_large() -> Workload:
    """RoBERTa-large shapes: 24 layers, hidden 1024, FFN 4096, vocab 50265, 514 positions."""
    d, ff, vocab = 1024, 4096, 50265
    ts = [_mat("emb.word", vocab, d, sparse_rows=0.9), _mat("emb.pos", 514, d), _mat("emb.type", 1, d),
          _vec("emb.ln.w", d, init="ones"), _vec("emb.ln.b", d)]
    for i in range(24):
        p = f"l{i}"
        for nm in ("q", "k", "v", "o"):
            ts += [_mat(f"{p}.{nm}.w", d, d), _vec(f"{p}.{nm}.b", d)]
        ts += [_mat(p + ".fc1.w", ff, d), _vec(p + ".fc1.b", ff), _mat(p + ".fc2.w", d, ff), _vec(p + ".fc2.b", d)]
        ts += [_vec(p + ".ln1.w", d, init="ones"), _vec(p + ".ln1.b", d),
               _vec(p + ".ln2.w", d, init="ones"), _vec(p + ".ln2.b", d)]
    ts += [_mat("head.dense.w", d, d), _vec("head.dense.b", d), _vec("head.ln.w", d, init="ones"),
           _vec("head.ln.b", d), _vec("head.bias", vocab)]
    return Workload("roberta_large", 2, tuple(ts), lr=1e-5, steps=20)


def llama_7b(layers: int = 32, vocab: int = 32000) -> Workload:
    """LLaMA-7B shapes: 32 layers, d 4096, SwiGLU FFN 11008, vocab 32000, RMSNorm; bf16 gradients."""
    d, ff = 4096, 11008
    ts = [_mat("embed", vocab, d)]
    for i in range(layers):
        p = f"l{i}"
        ts += [_mat(f"{p}.{nm}", d, d) for nm in ("q", "k", "v", "o")]
        ts += [_mat(p + ".gate", ff, d), _mat(p + ".up", ff, d), _mat(p + ".down", d, ff)]
        ts += [_vec(p + ".norm1", d, init="ones"), _vec(p + ".norm2", d, init="ones")]
    ts += [_vec("final_norm", d, init="ones"), _mat("lm_head", vocab, d)]
    name = "llama_7b" if (layers, vocab) == (32, 32000) else f"llama_7b_slice_{layers}l_{vocab}v"
    return Workload(name, 3, tuple(ts), lr=2e-5, weight_decay=0.0, grad_dtype="bf16", steps=20)


def llama_7b_flat() -> Workload:
    """The LLaMA-7B parameters packed into 1-D arrays, one per decoder layer plus embedding and head, as a
    sharded-data-parallel wrapper flattens them (App. D.2 "LLaMA": all parameters one-dimensional, hence block-wise
    normalization for both moments); bf16 gradients."""
    d, ff, vocab = 4096, 11008, 32000
    per_layer = 4 * d * d + 3 * d * ff + 2 * d
    ts = [_vec("embed", vocab * d)] + [_vec(f"l{i}", per_layer) for i in range(32)] + [_vec("head", vocab * d + d)]
    return Workload("llama_7b_flat", 5, tuple(ts), lr=2e-5, weight_decay=0.0, grad_dtype="bf16", steps=20)


def square_8192() -> Workload:
    """One 8192x8192 matrix for the quantizer/normalizer sweep."""
    return Workload("square_8192", 4, (_mat("weight", 8192, 8192),), lr=1e-3, steps=10)


def odd_shape(*dims) -> Workload:
    """One tensor of an awkward shape (rows that are not whole 128-blocks, or three / four axes such as a convolution
    weight), bf16 gradients: for timing the paths beside the tiled one."""
    rows = 1
    for d in dims[:-1]:
        rows *= d
    name = "x".join(str(d) for d in dims)
    spec = TensorSpec(name, rows, dims[-1], len(dims), dims=tuple(dims) if len(dims) >= 3 else None)
    return Workload("odd_" + name, 6, (spec,), lr=1e-3, grad_dtype="bf16", steps=10)


WORKLOADS = {
    "single_matrix": single_matrix,
    "transformer_base": transformer_base,
    "roberta_large": roberta_large,
    "llama_7b": llama_7b,
    "square_8192": square_8192,
    "llama_7b_flat": llama_7b_flat,
    # reduced LLaMA list (embedding, head and a few decoder layers) for profiler captures and quick checks
    "llama_7b_1l": lambda: llama_7b(layers=1),
    "llama_7b_4l": lambda: llama_7b(layers=4),
    # four decoder layers with a token table of 1024 rows: 0.82 G parameters, the matrices of the decoder alone
    "llama_7b_4l_1kv": lambda: llama_7b(layers=4, vocab=1024),
    "odd_8192x8200": lambda: odd_shape(8192, 8200),
    "odd_65536x1000": lambda: odd_shape(65536, 1000),
    "odd_8200x8193": lambda: odd_shape(8200, 8193),
    "odd_64x128x8192": lambda: odd_shape(64, 128, 8192),
    "odd_2048x2048x4x4": lambda: odd_shape(2048, 2048, 4, 4),
    "odd_4096x4096x3": lambda: odd_shape(4096, 4096, 3),
    "odd_1024x1000x3x3": lambda: odd_shape(1024, 1000, 3, 3),     # rows of whole lanes, not of whole blocks (9000 = 8 * 1125)
}


def tensor_seed(workload_index: int, tensor_index: int) -> int:
    return BASE_SEED + 1000 * workload_index + tensor_index


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_param(spec: TensorSpec, workload_index: int, tensor_index: int, device="cpu") -> torch.Tensor:
    """fp32 parameter tensor: matrices N(0, 0.02^2), norm weights 1, biases 0."""
    if spec.init == "ones":
        return torch.ones(spec.shape, dtype=torch.float32, device=device)
    if spec.init == "zeros":
        return torch.zeros(spec.shape, dtype=torch.float32, device=device)
    gen = _gen(device, tensor_seed(workload_index, tensor_index) + 7_000_000)
    return torch.randn(spec.shape, generator=gen, dtype=torch.float32, device=device) * 0.02


def make_grad(spec: TensorSpec, workload_index: int, tensor_index: int, step: int, device="cpu",
              dtype=torch.float32, outlier_p: float = 1e-3, out: torch.Tensor | None = None) -> torch.Tensor:
    """Gradient of `spec` at `step` (>= 1) following the module's recipe; returned in `dtype`."""
    seed = tensor_seed(workload_index, tensor_index)
    fixed = _gen(device, seed)                       # a_i, b_j, outlier positions: same every step
    fresh = _gen(device, seed + 100_000 * step)      # z: fresh every step
    rows, cols = spec.rows, spec.cols
    a = torch.exp(torch.randn(rows, 1, generator=fixed, dtype=torch.float32, device=device))
    g = torch.randn(rows, cols, generator=fresh, dtype=torch.float32, device=device)
    g *= a
    if spec.ndim >= 2:
        b = torch.exp(torch.randn(1, cols, generator=fixed, dtype=torch.float32, device=device))
        g *= b
    if outlier_p > 0:
        mask = torch.rand(rows, cols, generator=fixed, dtype=torch.float32, device=device) < outlier_p
        g = torch.where(mask, g * 100.0, g)
    if spec.sparse_rows > 0:
        keep = torch.rand(rows, 1, generator=fresh, dtype=torch.float32, device=device) >= spec.sparse_rows
        g = g * keep
    g = g.reshape(spec.shape).to(dtype)
    if out is not None:
        out.copy_(g)
        return out
    return g
