"""Seeded synthetic inputs shaped like BERT's fully-connected and embedding layers.

This module only draws random numbers; it contains none of the quantisation arithmetic, so both
the CUDA path and its CPU checker can be fed the same bytes from here.

Recipe (stands in for fine-tuned GLUE / SQuAD BERT tensors, which are not available offline):
  * weights, biases, embedding tables ~ N(0, 0.02)  (BERT's initialiser range);
  * activations ~ N(0, 1) ("after LayerNorm") with an i.i.d. Bernoulli(0.01) mask that multiplies
    entries by 8, so a few outliers set the per-tensor scale, as in real Transformer activations;
  * token ids uniform in [0, vocab).
Every tensor is drawn from numpy's counter-based Philox generator keyed by
``BASE_SEED + 1000 * config + tensor_index``.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 191006188
WEIGHT_SIGMA = 0.02
OUTLIER_PROB = 0.01
OUTLIER_GAIN = 8.0


def seed_for(config: int, tensor_index: int) -> int:
    return BASE_SEED + 1000 * int(config) + int(tensor_index)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed)))


def normal(shape, sigma: float, seed: int) -> np.ndarray:
    """fp32 tensor ~ N(0, sigma)."""
    x = _rng(seed).standard_normal(size=shape, dtype=np.float32)
    x *= np.float32(sigma)
    return x


def weight(n_out: int, k_in: int, seed: int) -> np.ndarray:
    """FC weight [N, K] (row-major, Y = X W^T) ~ N(0, 0.02)."""
    return normal((n_out, k_in), WEIGHT_SIGMA, seed)


def bias(n_out: int, seed: int) -> np.ndarray:
    return normal((n_out,), WEIGHT_SIGMA, seed)


def activation(m_tokens: int, k_in: int, seed: int) -> np.ndarray:
    """Activation [M, K] ~ N(0,1) with 1 % of entries multiplied by 8."""
    rng = _rng(seed)
    x = rng.standard_normal(size=(m_tokens, k_in), dtype=np.float32)
    mask = rng.random(size=(m_tokens, k_in), dtype=np.float32) < np.float32(OUTLIER_PROB)
    x[mask] *= np.float32(OUTLIER_GAIN)
    return x


def embedding_table(vocab: int, hidden: int, seed: int) -> np.ndarray:
    return normal((vocab, hidden), WEIGHT_SIGMA, seed)


def token_ids(count: int, vocab: int, seed: int) -> np.ndarray:
    return _rng(seed).integers(0, vocab, size=(count,), dtype=np.int32)


# (K, N, act) of the four quantised FC layers of one encoder block.
def fc_set(hidden: int, ffn: int):
    return [
        ("qkv", hidden, 3 * hidden, 0),
        ("attn_out", hidden, hidden, 0),
        ("ffn1", hidden, ffn, 1),
        ("ffn2", ffn, hidden, 0),
    ]


BERT_BASE = dict(hidden=768, ffn=3072, heads=12, layers=12, vocab=30522, max_pos=512, batch=32, seq=128)
BERT_LARGE = dict(hidden=1024, ffn=4096, heads=16, layers=24, vocab=30522, max_pos=512, batch=64, seq=384)
