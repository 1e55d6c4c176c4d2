"""CPU ORACLE of the sparse-attention consumer - TEST INFRASTRUCTURE ONLY.

What the consumer of the slot table computes (paper Sec. 2.1 "Top-k Sparse Attention": once the selected set is fixed,
attention is exact over the selected entries and unselected entries do not participate; Sec. 3.4 Phase 5: the
attention kernel reads the selected records out of the GPU cache through the emitted slots), written out as the plain
definition of softmax attention in fp64 numpy, for the record layout of the DSA configurations: a record is D bf16
numbers (E = 2 D bytes; D = 576 = a 512-number compressed latent followed by a 64-number rotary key); the key of a
record is all D numbers, its value the first Dv of them (the absorbed form of multi-head latent attention: per head
the query is a D-vector, scores are dot products with the whole record, the output is a weighted sum of the latents).

    out[n, h, :] = sum_j p[n, h, j] * value(rec[n, j]),   p[n, h, :] = softmax_j(scale * q[n, h, :] . key(rec[n, j]))
    lse[n, h]    = log sum_j exp(scale * q[n, h, :] . key(rec[n, j]))

over the entries j whose slot-table value is >= 0 (a -1 entry is padding and takes no part); a row with no valid entry
gives out = 0 and lse = -inf.  rec[n, j] = the E bytes at record index table[n, j] of the layer's pool.

Nothing on the product path may import this file; it shares no code with the CUDA library.
Pins (tests/test_attention_oracle.py): equal keys give the mean of the values, one dominant key gives its own value,
the weights and lse against scipy's softmax / logsumexp on the same scores, invariance under a change of placement
(the paper's exactness property), invariance under the order of the selections, padding ignored, and the additive
decomposition over splits of the selection that a split-k kernel relies on.
"""
from __future__ import annotations

import numpy as np


def bf16_to_f64(raw: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bfloat16 numbers -> float64 (bf16 is the upper half of an IEEE float32)."""
    raw = np.ascontiguousarray(raw, dtype=np.uint16)
    return (raw.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (round to nearest even), for building test inputs."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (b + 0x7FFF + ((b >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def sparse_attention(pool: np.ndarray, table: np.ndarray, q_bf16: np.ndarray, value_dims: int, scale: float):
    """pool: uint8 [records][E]; table: int32 [N][k] record indices or -1; q_bf16: uint16 [N][H][D] bf16 bit patterns.
    Returns (out float64 [N][H][value_dims], lse float64 [N][H])."""
    pool = np.ascontiguousarray(pool, dtype=np.uint8)
    table = np.asarray(table)
    N, k = table.shape
    E = pool.shape[1]
    D = E // 2
    H = q_bf16.shape[1]
    assert q_bf16.shape == (N, H, D) and value_dims <= D
    q = bf16_to_f64(q_bf16)
    out = np.zeros((N, H, value_dims), dtype=np.float64)
    lse = np.full((N, H), -np.inf, dtype=np.float64)
    for n in range(N):
        idx = table[n][table[n] >= 0]
        if idx.size == 0:
            continue
        rec = bf16_to_f64(pool[idx].reshape(-1).view(np.uint16)).reshape(idx.size, D)
        s = scale * (q[n] @ rec.T)                           # [H][valid]
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(axis=1, keepdims=True)
        out[n] = (e / z) @ rec[:, :value_dims]
        lse[n] = (m + np.log(z))[:, 0]
    return out, lse
