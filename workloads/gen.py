"""Seeded, counter-based synthetic inputs for the MoE-FFN layer.

This module is the only code shared by the CPU oracle's tests and the CUDA
path's tests/bench.  It holds none of the layer's arithmetic: it only draws
numbers.  Every value is a pure function of (seed, tensor id, element index),
so any slice of any tensor can be regenerated on any device, in any order,
and comes out bit-identical on CPU and on GPU (integer hashing, one exact
int->fp32 conversion, one IEEE fp32 multiply, one round-to-nearest-even to
bf16 -- no transcendental functions).

Distribution: each element is the centred sum of eight independent 16-bit
uniforms (Irwin-Hall, n = 8) scaled to the requested standard deviation.
That is a close stand-in for a normal law (excess kurtosis -0.15, support
+-4.9 sigma); the layer's cost and numerics do not depend on the tails.
"""
from __future__ import annotations

import math

import torch

# tensor ids (the "stream" of the counter-based generator)
TID_X, TID_W_GATE_UP, TID_W_DOWN, TID_W_ROUTER, TID_DOUT, TID_PERM, TID_MISC = 1, 2, 3, 4, 5, 6, 7

_M64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Python int (mod 2^64) -> the same bit pattern as a signed 64-bit value."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


_C_GOLD = _s64(0x9E3779B97F4A7C15)
_C_MUL1 = _s64(0xBF58476D1CE4E5B9)
_C_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 lanes."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    """SplitMix64 output function on int64 lanes (wrap-around arithmetic)."""
    z = (z ^ _lsr(z, 30)) * _C_MUL1
    z = (z ^ _lsr(z, 27)) * _C_MUL2
    return z ^ _lsr(z, 31)


def mix64_py(z: int) -> int:
    """Same function on a Python int; used by the tests to pin the tensor version."""
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, tid: int) -> int:
    """64-bit key of one tensor's stream."""
    return mix64_py(mix64_py(seed * 0x9E3779B97F4A7C15 + 0x1234567) ^ (tid * 0xD1B54A32D192ED03))


def hash_u64(seed: int, tid: int, idx: torch.Tensor) -> torch.Tensor:
    """Hash of element indices `idx` (int64 tensor) under stream (seed, tid); int64 bit patterns."""
    key = _s64(stream_key(seed, tid))
    return _mix64(idx * _C_GOLD + key)


_IH_N = 8
# std of (2*sum_of_8_u16 - 8*65535): each 2*u has variance 4*(65536^2-1)/12
_IH_STD = math.sqrt(_IH_N * 4.0 * (65536.0 ** 2 - 1.0) / 12.0)


def normal_f32(seed: int, tid: int, start: int, count: int, std: float, device="cpu",
               chunk: int = 1 << 24) -> torch.Tensor:
    """`count` fp32 values of stream (seed, tid) starting at element `start`; std `std`."""
    out = torch.empty(count, dtype=torch.float32, device=device)
    scale = torch.tensor(std / _IH_STD, dtype=torch.float32).item()  # one fp32 constant
    for c0 in range(0, count, chunk):
        n = min(chunk, count - c0)
        idx = torch.arange(start + c0, start + c0 + n, dtype=torch.int64, device=device)
        acc = torch.zeros(n, dtype=torch.int64, device=device)
        for half in range(2):
            h = hash_u64(seed, tid, idx * 2 + half)
            for f in range(4):
                acc += _lsr(h, 16 * f) & 0xFFFF
        centred = (acc * 2 - _IH_N * 65535).to(torch.float32)  # |.| < 2^24: exact
        out[c0:c0 + n] = centred * scale
    return out


def normal_bf16(seed: int, tid: int, shape, std: float, device="cpu", start: int = 0) -> torch.Tensor:
    """bf16 tensor of `shape` from stream (seed, tid), elements start..start+numel-1."""
    n = 1
    for s in shape:
        n *= int(s)
    return normal_f32(seed, tid, start, n, std, device).to(torch.bfloat16).reshape(*shape)


def permutation(seed: int, tid: int, n: int) -> torch.Tensor:
    """Seeded permutation of range(n) (CPU int64): argsort of hashed keys, ties by index."""
    h = hash_u64(seed, tid, torch.arange(n, dtype=torch.int64))
    return torch.argsort(h, stable=True)
