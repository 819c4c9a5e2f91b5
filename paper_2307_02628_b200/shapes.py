"""The model description the binding takes: layer count, widths, vocabulary, storage type."""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int
    max_pos: int
    dtype: str  # "fp32" | "bf16": storage type of weights, GEMM operands and KV cache

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads


def storage_dtype(shape: ModelShape) -> torch.dtype:
    return torch.float32 if shape.dtype == "fp32" else torch.bfloat16
