"""Counter-based input generator (numpy), bit-reproducible on any machine.

Definition (every step is integer arithmetic mod 2**64 or a single IEEE-754
binary32 operation, so an independent implementation reproduces every bit):

* ``splitmix64_at(seed, c)`` is output number ``c + 1`` of the SplitMix64
  generator (Steele, Lea, Flood 2014) started from state ``seed``::

      z = seed + (c + 1) * 0x9E3779B97F4A7C15
      z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9
      z = (z ^ (z >> 27)) * 0x94D049BB133111EB
      return z ^ (z >> 31)

* row ``k`` of a matrix drawn with seed ``seed`` has the key
  ``row_key = splitmix64_at(seed, k)``.
* element ``i`` of that row takes the two words
  ``h0 = splitmix64_at(row_key, 2 i)`` and ``h1 = splitmix64_at(row_key, 2 i + 1)``,
  adds their eight 16-bit fields into ``S`` (0 .. 8 * 65535), and returns the
  Irwin-Hall approximation of a standard normal
  ``x = float32(S - 262140) * INV_SIGMA_F32`` (one rounding), where
  ``INV_SIGMA_F32 = float32(1 / sqrt(8 * (2**32 - 1) / 12))``.
* a value with mean ``m`` and standard deviation ``sd`` is
  ``fl32(fl32(x * sd) + m)`` (two roundings, never a fused multiply-add).

The sum of eight uniforms has excess kurtosis -0.15 and support +-4.9 sigma:
close enough to the N(0,1) gradients the workloads call for, and exactly
reproducible, which a libm-based Box-Muller is not.
"""
from __future__ import annotations

import numpy as np

ADV_REVGRAD = 0  # received row replaced by -c * (honest row)
ADV_CONST = 1    # received row replaced by kappa * ones
ADV_GAUSS = 2    # received row += sigma * noise

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_MASK16 = np.uint64(0xFFFF)

IH_CENTER = 4 * 65535  # mean of the sum of eight 16-bit uniforms
INV_SIGMA_F32 = np.float32(1.0 / np.sqrt(8.0 * (2.0 ** 32 - 1.0) / 12.0))


def splitmix64_at(seed, ctr):
    """Output number ``ctr + 1`` of SplitMix64 started at ``seed`` (vectorised)."""
    with np.errstate(over="ignore"):
        z = np.uint64(seed) + (np.asarray(ctr, dtype=np.uint64) + np.uint64(1)) * _GAMMA
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def row_key(seed: int, row: int) -> np.uint64:
    return np.uint64(splitmix64_at(np.uint64(seed & 0xFFFFFFFFFFFFFFFF), np.uint64(row)))


def _sum16(h):
    s = (h & _MASK16) + ((h >> np.uint64(16)) & _MASK16)
    s += (h >> np.uint64(32)) & _MASK16
    s += h >> np.uint64(48)
    return s


_BLOCK = 1 << 16  # elements per pass: keeps the temporaries cache-resident


def approx_normal_at(seed: int, row: int, idx) -> np.ndarray:
    """Standard-normal-like float32 values of row ``row`` at coordinates ``idx``."""
    idx = np.asarray(idx, dtype=np.uint64)
    key = row_key(seed, row)
    out = np.empty(idx.shape[0], dtype=np.float32)
    for b0 in range(0, idx.shape[0], _BLOCK):
        part = idx[b0:b0 + _BLOCK]
        with np.errstate(over="ignore"):
            c0 = part * np.uint64(2)
            s = _sum16(splitmix64_at(key, c0)) + _sum16(splitmix64_at(key, c0 + np.uint64(1)))
        centred = s.astype(np.int64) - np.int64(IH_CENTER)
        out[b0:b0 + _BLOCK] = centred.astype(np.float32) * INV_SIGMA_F32
    return out


def approx_normal_rows(seed: int, rows, i0: int, i1: int, mean: float = 0.0, std: float = 1.0,
                       idx=None) -> np.ndarray:
    """float32 ``[len(rows)][i1 - i0]`` (or ``[len(rows)][len(idx)]``) with the given mean / std."""
    if idx is None:
        idx = np.arange(i0, i1, dtype=np.uint64)
    rows = list(rows)
    out = np.empty((len(rows), len(idx)), dtype=np.float32)
    sd = np.float32(std)
    mu = np.float32(mean)
    for r, k in enumerate(rows):
        x = approx_normal_at(seed, int(k), idx)
        out[r] = (x * sd) + mu
    return out


def gradient_rows(seed: int, n: int, d: int, mean: float = 0.0, std: float = 1.0,
                  i0: int = 0, i1: int | None = None, idx=None) -> np.ndarray:
    """Per-partition gradients ``G[n][.]`` (float32): row k = gradient g_k."""
    if i1 is None:
        i1 = d
    return approx_normal_rows(seed, range(n), i0, i1, mean, std, idx)


def projection_vector(seed: int, d: int, i0: int = 0, i1: int | None = None, idx=None) -> np.ndarray:
    """The locator's random vector f (mean 1, variance 1), float32 ``[.]``."""
    if i1 is None:
        i1 = d
    return approx_normal_rows(seed, [0], i0, i1, 1.0, 1.0, idx)[0]


def complex_rows(seed: int, n: int, d: int, std: float = 1.0, i0: int = 0, i1: int | None = None,
                 idx=None) -> np.ndarray:
    """A synthetic complex64 matrix ``[n][.]``: element i of a row is
    (value 2 i) + 1j * (value 2 i + 1) of the real generator over 2 d values."""
    if i1 is None:
        i1 = d
    if idx is None:
        flat = approx_normal_rows(seed, range(n), 2 * i0, 2 * i1, 0.0, std)
    else:
        idx = np.asarray(idx, dtype=np.uint64)
        both = np.stack([idx * np.uint64(2), idx * np.uint64(2) + np.uint64(1)], axis=1).reshape(-1)
        flat = approx_normal_rows(seed, range(n), 0, 0, 0.0, std, idx=both)
    return np.ascontiguousarray(flat).view(np.complex64)


def choose_adversaries(seed: int, n: int, count: int) -> np.ndarray:
    """``count`` distinct worker indices, uniformly at random, ascending."""
    rng = np.random.default_rng(seed)
    return np.sort(rng.choice(n, size=count, replace=False)).astype(np.int32)


def apply_adversaries(R: np.ndarray, adv_idx, adv_model, adv_param, seed: int,
                      i0: int = 0, idx=None) -> np.ndarray:
    """Corrupt rows ``adv_idx`` of the received matrix in place and return it.

    ``R`` is float32 ``[n][L]`` or complex64 ``[n][L]``; a complex matrix is
    treated as its interleaved float32 view (2 L values per row).  ``i0`` (or
    ``idx``) gives the coordinates the columns of ``R`` stand for, so a slice
    or a sample of a large matrix is corrupted exactly as the whole would be.

    * ``ADV_REVGRAD``: row <- fl32(row * (-c))
    * ``ADV_CONST``  : row <- kappa (imaginary parts 0 for a complex matrix)
    * ``ADV_GAUSS``  : row <- fl32(row + fl32(x * sigma)), x from the generator
      with seed ``seed`` and row index = the worker index
    """
    is_complex = np.iscomplexobj(R)
    V = R.view(np.float32) if is_complex else R
    L = R.shape[1]
    if idx is None:
        cidx = np.arange(i0, i0 + L, dtype=np.uint64)
    else:
        cidx = np.asarray(idx, dtype=np.uint64)
    if is_complex:
        fidx = np.stack([cidx * np.uint64(2), cidx * np.uint64(2) + np.uint64(1)], axis=1).reshape(-1)
    else:
        fidx = cidx
    for j, model, param in zip(adv_idx, adv_model, adv_param):
        j = int(j)
        p = np.float32(param)
        if model == ADV_REVGRAD:
            V[j] = V[j] * np.float32(-p)
        elif model == ADV_CONST:
            if is_complex:
                V[j, 0::2] = p
                V[j, 1::2] = np.float32(0.0)
            else:
                V[j] = p
        elif model == ADV_GAUSS:
            x = approx_normal_at(seed, j, fidx)
            V[j] = V[j] + (x * p)
        else:
            raise ValueError(f"unknown adversary model {model}")
    return R
