"""Seeded synthetic inputs shared by the tests, the oracle checks and the benchmark.

This module holds none of the method's arithmetic: it only produces bytes.
Every value is a pure function of (seed, element index) through a counter-based
generator (the splitmix64 finaliser applied to ``seed + (index+1)*golden``), so
any sub-range can be regenerated independently and the CPU oracle and the GPU
path always read identical operands.

The tensors stand in for the ImageNet activations / SST-2 token embeddings and
the trained ResNet-50 v1.5 / BERT weights that the paper's evaluation used:
same shapes, plausible value distributions, no dataset needed.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _mix64(idx: np.ndarray, seed: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = (idx + np.uint64(1)) * _GOLDEN + np.uint64(seed & 0xFFFFFFFFFFFFFFFF)
        z ^= z >> np.uint64(30)
        z *= _M1
        z ^= z >> np.uint64(27)
        z *= _M2
        z ^= z >> np.uint64(31)
    return z


def _fill(out: np.ndarray, convert, start: int = 0) -> np.ndarray:
    """out[i] = convert(hash words of element indices start+i), chunk by chunk.  Every element is a
    pure function of its own index, so large arrays are filled by a few threads at once (NumPy
    releases the interpreter lock inside its loops) with the same result as a serial fill."""
    count = out.size

    def one(pos: int) -> None:
        n = min(_CHUNK, count - pos)
        out[pos:pos + n] = convert(np.arange(start + pos, start + pos + n, dtype=np.uint64))

    starts = range(0, count, _CHUNK)
    workers = min(len(starts), _THREADS)
    if workers <= 1:
        for pos in starts:
            one(pos)
    else:
        with ThreadPoolExecutor(max_workers=workers) as pool:
            list(pool.map(one, starts))
    return out


_THREADS = max(1, min(16, os.cpu_count() or 1))


def raw_u64(count: int, seed: int, start: int = 0) -> np.ndarray:
    """``count`` 64-bit hash words for element indices start .. start+count-1."""
    return _fill(np.empty(count, dtype=np.uint64), lambda idx: _mix64(idx, seed), start)


def uniform_s8(count: int, seed: int) -> np.ndarray:
    """int8 uniform over [-128, 127]."""
    return _fill(np.empty(count, dtype=np.int8),
                 lambda idx: (_mix64(idx, seed) & np.uint64(0xFF)).astype(np.uint8).view(np.int8))


def uniform_u8(count: int, seed: int) -> np.ndarray:
    """uint8 uniform over [0, 255] (post-ReLU activations)."""
    return _fill(np.empty(count, dtype=np.uint8), lambda idx: (_mix64(idx, seed) & np.uint64(0xFF)).astype(np.uint8))


def normal_s8(count: int, seed: int, sigma: float, lo: int = -128, hi: int = 127) -> np.ndarray:
    """int8 values round(sigma * z), z standard normal (Box-Muller on the two
    32-bit halves of the hash word), clipped to [lo, hi]."""
    def convert(idx):
        h = _mix64(idx, seed)
        u1 = ((h >> np.uint64(32)).astype(np.float64) + 1.0) / 4294967296.0
        u2 = (h & np.uint64(0xFFFFFFFF)).astype(np.float64) / 4294967296.0
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        return np.clip(np.rint(sigma * z), lo, hi).astype(np.int8)
    return _fill(np.empty(count, dtype=np.int8), convert)


def uniform_s32(count: int, seed: int, bound: int = 1 << 20) -> np.ndarray:
    """int32 uniform over [-bound, bound] (seeded C for accumulate=1 runs)."""
    span = np.uint64(2 * bound + 1)
    return _fill(np.empty(count, dtype=np.int32),
                 lambda idx: ((_mix64(idx, seed) >> np.uint64(11)) % span).astype(np.int64) - bound)


def seed_for(config_index: int, operand_id: int) -> int:
    """Seed convention: 0x11728 + 1000*config + operand (A=1, B=2, C=3)."""
    return 0x11728 + 1000 * config_index + operand_id


# ---------------------------------------------------------------------------
# Shape tables of the synthetic workloads (shapes only, no arithmetic).
# ---------------------------------------------------------------------------

#: ResNet-50 v1.5 convolutions: (count, H, W, Cin, Cout, R, S, stride, pad); stride sits
#: on the 3x3 of each down-sampling bottleneck.  23 distinct shapes, 53 layers.
RESNET50_CONVS = [
    (1, 224, 224, 3, 64, 7, 7, 2, 3),
    (1, 56, 56, 64, 64, 1, 1, 1, 0),
    (3, 56, 56, 64, 64, 3, 3, 1, 1),
    (4, 56, 56, 64, 256, 1, 1, 1, 0),
    (2, 56, 56, 256, 64, 1, 1, 1, 0),
    (1, 56, 56, 256, 128, 1, 1, 1, 0),
    (1, 56, 56, 128, 128, 3, 3, 2, 1),
    (4, 28, 28, 128, 512, 1, 1, 1, 0),
    (1, 56, 56, 256, 512, 1, 1, 2, 0),
    (3, 28, 28, 512, 128, 1, 1, 1, 0),
    (3, 28, 28, 128, 128, 3, 3, 1, 1),
    (1, 28, 28, 512, 256, 1, 1, 1, 0),
    (1, 28, 28, 256, 256, 3, 3, 2, 1),
    (6, 14, 14, 256, 1024, 1, 1, 1, 0),
    (1, 28, 28, 512, 1024, 1, 1, 2, 0),
    (5, 14, 14, 1024, 256, 1, 1, 1, 0),
    (5, 14, 14, 256, 256, 3, 3, 1, 1),
    (1, 14, 14, 1024, 512, 1, 1, 1, 0),
    (1, 14, 14, 512, 512, 3, 3, 2, 1),
    (3, 7, 7, 512, 2048, 1, 1, 1, 0),
    (1, 14, 14, 1024, 2048, 1, 1, 2, 0),
    (2, 7, 7, 2048, 512, 1, 1, 1, 0),
    (2, 7, 7, 512, 512, 3, 3, 1, 1),
]

#: Encoder GEMMs as (name, N, K); M is the token count T = batch * seq.
BERT_GEMMS = [
    ("base_qkv", 2304, 768),
    ("base_attn_out", 768, 768),
    ("base_ffn1", 3072, 768),
    ("base_ffn2", 768, 3072),
    ("large_qkv", 3072, 1024),
    ("large_ffn1", 4096, 1024),
    ("large_ffn2", 1024, 4096),
]
BERT_TOKENS = [8 * 128, 8 * 512, 32 * 512]

#: Decode-style weight matrices (N, K) and token counts M.
SKINNY_WEIGHTS = [(4096, 4096), (11008, 4096), (4096, 11008), (14336, 4096)]
SKINNY_M = [1, 4, 8, 16]

#: Square sweep sizes.
SQUARE_SIZES = [1024, 2048, 4096, 8192, 16384]
