"""Seeded synthetic inputs shaped like the paper's LLM-layer workloads (Table 1).

This module is the only code that serves both the CUDA path and the CPU oracle.
It holds none of the method's arithmetic: it draws numbers, converts them once to
the storage type and places probe values.  Everything is a pure function of its
seed.  bf16 tensors are produced as ``uint16`` bit patterns (numpy) so that the
same bytes reach both sides; ``to_torch`` reinterprets them without a copy.

The second parameter of every N(., .) is a standard deviation.
"""
from __future__ import annotations

import numpy as np


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed)))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Storage conversion binary32 -> bf16 (round to nearest even), as uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)
    return r


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def f32_to_f8e4m3_bits(x: np.ndarray) -> np.ndarray:
    """Storage conversion binary32 -> 8-bit float e4m3 (torch's round to nearest even), as uint8 bits."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.float8_e4m3fn)
    return t.view(torch.uint8).numpy()


def f8e4m3_bits_to_f32(b: np.ndarray) -> np.ndarray:
    import torch
    return torch.from_numpy(np.ascontiguousarray(b, dtype=np.uint8)).view(torch.float8_e4m3fn).to(torch.float32).numpy()


def normal_f8e4m3(shape, std: float, seed: int, mean: float = 0.0) -> np.ndarray:
    return f32_to_f8e4m3_bits(normal_f32(shape, std, seed, mean))


def int_valued_f8e4m3(shape, lo: int, hi: int, seed: int) -> np.ndarray:
    """Integers in [lo, hi] (|v| <= 16 are exact in e4m3)."""
    v = _rng(seed).integers(lo, hi + 1, size=shape)
    return f32_to_f8e4m3_bits(v.astype(np.float32))


def normal_f32(shape, std: float, seed: int, mean: float = 0.0) -> np.ndarray:
    g = _rng(seed).standard_normal(size=shape, dtype=np.float64)
    return (g * std + mean).astype(np.float32)


def normal_bf16(shape, std: float, seed: int, mean: float = 0.0) -> np.ndarray:
    return f32_to_bf16_bits(normal_f32(shape, std, seed, mean))


def uniform_bf16(shape, lo: float, hi: float, seed: int) -> np.ndarray:
    u = _rng(seed).random(size=shape, dtype=np.float64) * (hi - lo) + lo
    return f32_to_bf16_bits(u.astype(np.float32))


def int_valued_bf16(shape, lo: int, hi: int, seed: int) -> np.ndarray:
    """Integers in [lo, hi] (|v| <= 256 are exact in bf16)."""
    v = _rng(seed).integers(lo, hi + 1, size=shape)
    return f32_to_bf16_bits(v.astype(np.float32))


def spread_exponents_bf16(bits: np.ndarray, seed: int, lo: int = -20, hi: int = 20) -> np.ndarray:
    """Second draw of an input set: every element times 2^e, e uniform in [lo, hi]
    (App. E: narrow exponents hide a regrouping).  Exact: only the exponent moves."""
    e = _rng(seed).integers(lo, hi + 1, size=bits.shape)
    f = bf16_bits_to_f32(bits) * np.exp2(e).astype(np.float32)
    return f32_to_bf16_bits(f)


def spread_exponents_f32(x: np.ndarray, seed: int, lo: int = -20, hi: int = 20) -> np.ndarray:
    e = _rng(seed).integers(lo, hi + 1, size=x.shape)
    return (x * np.exp2(e).astype(np.float32)).astype(np.float32)


def add_cancellation_pairs(x: np.ndarray, seed: int, pairs: int = 64, mag: float = 1e8) -> np.ndarray:
    """On even rows, overwrite `pairs` disjoint random position pairs with (+mag, -mag).
    1e8 is exact in binary32."""
    x = np.array(x, dtype=np.float32, copy=True)
    R, Cc = x.shape
    g = _rng(seed)
    for r in range(0, R, 2):
        pos = g.choice(Cc, size=2 * pairs, replace=False)
        x[r, pos[:pairs]] = np.float32(mag)
        x[r, pos[pairs:]] = np.float32(-mag)
    return x


def lr_probe_row(K: int, r_at: int, plus_at: int, minus_at: int, L: float = 1024.0,
                 r: float = 2.0 ** -15) -> np.ndarray:
    """The +L / -L / r probe row of Sec. 4: an otherwise empty axis."""
    v = np.zeros(K, dtype=np.float32)
    v[r_at] = r
    v[plus_at] = L
    v[minus_at] = -L
    return v


def to_torch(a: np.ndarray, device="cpu"):
    """numpy -> torch without changing a bit; uint16 arrays become torch.bfloat16."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.to(device)


def from_torch(t) -> np.ndarray:
    """torch -> numpy; bfloat16 tensors come back as uint16 bit patterns."""
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.uint16).numpy() if hasattr(torch, "uint16") else t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


# ---------------------------------------------------------------- device-side draws
# Full-size tensors (up to 8 GiB) are drawn on the GPU with torch's counter-based generator;
# the oracle then reads back the rows it checks, so both sides still see the same bytes.
def device_normal(shape, std: float, seed: int, dtype, device="cuda", mean: float = 0.0, chunk_rows: int = 4096):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    out = torch.empty(shape, dtype=dtype, device=device)
    rows = shape[0]
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        blk = torch.randn((r1 - r0,) + tuple(shape[1:]), generator=g, device=device, dtype=torch.float32)
        out[r0:r1] = (blk * std + mean).to(dtype)
    return out


def device_uniform(shape, lo: float, hi: float, seed: int, dtype, device="cuda"):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    u = torch.rand(shape, generator=g, device=device, dtype=torch.float32)
    return (u * (hi - lo) + lo).to(dtype)


def device_add_cancellation_pairs(x, seed: int, pairs: int = 64, mag: float = 1e8):
    """In place: on even rows, `pairs` disjoint positions get +mag and `pairs` others -mag.
    Positions are (base + stride * t) mod C with an odd stride, a bijection when C is a power
    of two, so the 2*pairs positions of a row are distinct."""
    import torch
    R, Cc = x.shape
    assert Cc & (Cc - 1) == 0 and 2 * pairs <= Cc
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    rows = torch.arange(0, R, 2)
    base = torch.randint(0, Cc, (rows.numel(), 1), generator=g)
    stride = torch.randint(0, Cc // 2, (rows.numel(), 1), generator=g) * 2 + 1
    t = torch.arange(2 * pairs).unsqueeze(0)
    pos = ((base + stride * t) % Cc).to(x.device)
    vals = torch.cat([torch.full((pairs,), mag), torch.full((pairs,), -mag)]).to(x.dtype).to(x.device)
    x[rows.to(x.device).unsqueeze(1), pos] = vals.unsqueeze(0).expand(rows.numel(), -1)
    return x
