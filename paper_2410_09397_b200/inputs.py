"""Seeded synthetic inputs for exact softmax attention (Q, K, V, dO, block masks).

This module holds only input generation: a counter-based random number stream,
the bf16 storage conversion, and the table of benchmark workloads.  It contains
none of the attention arithmetic, so both the CPU oracle's tests and the CUDA
path's tests can draw the very same bits from it.

Generator (all integer arithmetic modulo 2**64):

* ``splitmix64`` finaliser (Steele, Lea & Flood 2014, "Fast splittable
  pseudorandom number generators"): ``z ^= z >> 30; z *= 0xBF58476D1CE4E5B9;
  z ^= z >> 27; z *= 0x94D049BB133111EB; z ^= z >> 31``.
* stream ``s`` has base ``mix(s * GOLDEN + 1)``; its ``k``-th 64-bit word is
  ``mix(base + (k + 1) * GOLDEN)`` with ``GOLDEN = 0x9E3779B97F4A7C15``.
* a uniform in (0, 1) is ``((word >> 11) + 0.5) / 2**53``.
* element ``e`` of a normal tensor uses words ``2e`` and ``2e + 1`` in the
  Box-Muller transform ``sqrt(-2 ln u1) * cos(2 pi u2)``, evaluated in float64
  and then rounded to float32 (and, for bf16 workloads, to bf16 with
  round-to-nearest-even).

Every element is addressable by its index, so a slice of a tensor (one head of a
large workload) can be generated without generating the rest.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# tensor ids inside one workload seed
TENSOR_Q, TENSOR_K, TENSOR_V, TENSOR_DO, TENSOR_AUX = 0, 1, 2, 3, 4

MASK_NONE, MASK_CAUSAL, MASK_BLOCK_SPARSE, MASK_BLOCK_SPARSE_CAUSAL, MASK_ELEMENT = 0, 1, 2, 3, 4


def is_block_mask(kind: int) -> bool:
    return kind in (MASK_BLOCK_SPARSE, MASK_BLOCK_SPARSE_CAUSAL)


def _mix(z: np.ndarray) -> np.ndarray:
    z = z ^ (z >> np.uint64(30))
    z = z * _M1
    z = z ^ (z >> np.uint64(27))
    z = z * _M2
    return z ^ (z >> np.uint64(31))


def stream_words(stream: int, start: int, count: int) -> np.ndarray:
    """Words ``start .. start+count-1`` of stream ``stream`` as uint64."""
    with np.errstate(over="ignore"):
        base = _mix(np.uint64(stream) * GOLDEN + np.uint64(1))
        k = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        return _mix(base + k * GOLDEN)


def uniform(stream: int, start: int, count: int) -> np.ndarray:
    """``count`` float64 uniforms in (0, 1), one word each, from word ``start``."""
    w = stream_words(stream, start, count)
    return ((w >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal_f32(stream: int, start: int, count: int, chunk: int = 1 << 22) -> np.ndarray:
    """Elements ``start .. start+count-1`` of the N(0,1) tensor of ``stream`` (float32)."""
    out = np.empty(count, dtype=np.float32)
    done = 0
    while done < count:
        c = min(chunk, count - done)
        u = uniform(stream, 2 * (start + done), 2 * c)
        u1, u2 = u[0::2], u[1::2]
        out[done:done + c] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
        done += c
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even); returns the uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return ((b + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 values rounded to the nearest bf16, returned as float32."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


def stream_id(seed: int, tensor_id: int) -> int:
    return seed * 8 + tensor_id


def normal_tensor(seed: int, tensor_id: int, shape, *, bf16: bool, start: int = 0) -> np.ndarray:
    """N(0,1) tensor of the given shape (float32 values; bf16-representable if ``bf16``).

    ``start`` is the flat element offset inside the full tensor of that stream,
    so a head of a big workload is ``start = (b * heads + h) * n * d``.
    """
    count = int(np.prod(shape))
    x = normal_f32(stream_id(seed, tensor_id), start, count)
    if bf16:
        x = round_to_bf16(x)
    return x.reshape(shape)


def block_mask(seed: int, n_blocks: int, keep_prob: float, heads: int = 1) -> np.ndarray:
    """uint8 ``[heads, n_blocks, n_blocks]``: 1 on the diagonal, else 1 with probability ``keep_prob``.

    Row-major draw order, one uniform per block (diagonal blocks consume theirs too).
    """
    u = uniform(stream_id(seed, TENSOR_AUX), 0, heads * n_blocks * n_blocks)
    m = (u < keep_prob).reshape(heads, n_blocks, n_blocks)
    eye = np.eye(n_blocks, dtype=bool)[None]
    return (m | eye).astype(np.uint8)


def element_mask(seed: int, n: int, keep_prob: float, heads: int = 1) -> np.ndarray:
    """uint8 ``[heads, n, n]``: every entry kept with probability ``keep_prob`` (row-major draw order)."""
    u = uniform(stream_id(seed, TENSOR_AUX), 0, heads * n * n)
    return (u < keep_prob).reshape(heads, n, n).astype(np.uint8)


def pack_element_mask(keep: np.ndarray) -> np.ndarray:
    """Keep matrix ``[heads, n, n]`` -> int32 bitmap ``[heads, n, ceil(n / 32)]``: bit j % 32 of word j / 32."""
    h, n, _ = keep.shape
    words = (n + 31) // 32
    padded = np.zeros((h, n, words * 32), dtype=np.uint8)
    padded[:, :, :n] = keep != 0
    bits = np.packbits(padded.reshape(h, n, words, 32), axis=-1, bitorder="little")   # 4 bytes per word, low bits first
    return np.ascontiguousarray(bits).view("<u4").reshape(h, n, words).astype(np.uint32).view(np.int32)


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shape, storage type, mask)."""

    name: str
    batch: int
    heads: int
    n: int
    d: int
    dtype: str          # "f32" or "bf16"
    mask: int           # MASK_*
    seed: int
    block: int = 128
    keep_prob: float = 0.1
    mask_seed: int = 5

    @property
    def bf16(self) -> bool:
        return self.dtype == "bf16"

    def kept_entries_per_head(self, bmask: np.ndarray | None = None) -> int:
        if self.mask == MASK_NONE:
            return self.n * self.n
        if self.mask == MASK_CAUSAL:
            return self.n * (self.n + 1) // 2
        assert bmask is not None
        if self.mask == MASK_BLOCK_SPARSE_CAUSAL:   # whole blocks below the diagonal, kept diagonal blocks with j <= i
            m = bmask[0].astype(bool)
            return int(np.tril(m, -1).sum()) * self.block * self.block + int(np.diag(m).sum()) * (self.block * (self.block + 1) // 2)
        return int(bmask[0].sum()) * self.block * self.block

    def tensors(self, head_slice: tuple[int, int] | None = None) -> dict[str, np.ndarray]:
        """Q, K, V, dO as float32 ``[B*H (or slice), n, d]`` arrays of this workload.

        ``head_slice=(lo, hi)`` generates only flattened (batch, head) indices ``lo..hi-1``.
        """
        bh = self.batch * self.heads
        lo, hi = (0, bh) if head_slice is None else head_slice
        per = self.n * self.d
        out = {}
        for name, tid in (("Q", TENSOR_Q), ("K", TENSOR_K), ("V", TENSOR_V), ("dO", TENSOR_DO)):
            out[name] = normal_tensor(self.seed, tid, (hi - lo, self.n, self.d), bf16=self.bf16, start=lo * per)
        return out

    def block_mask(self) -> np.ndarray | None:
        if not is_block_mask(self.mask):
            return None
        nb = (self.n + self.block - 1) // self.block
        return block_mask(self.mask_seed, nb, self.keep_prob, heads=1)


WORKLOADS = {
    "C1": Workload("C1", 1, 1, 128, 64, "f32", MASK_NONE, seed=0),
    "C2": Workload("C2", 4, 16, 2048, 64, "bf16", MASK_NONE, seed=1),
    "C3": Workload("C3", 2, 16, 8192, 128, "bf16", MASK_CAUSAL, seed=2),
    "C4": Workload("C4", 1, 8, 4096, 256, "bf16", MASK_NONE, seed=3),
    "C5": Workload("C5", 1, 32, 32768, 128, "bf16", MASK_BLOCK_SPARSE, seed=4),
}
