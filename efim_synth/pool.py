"""Counter-based fill of the paged KV pools.

Every element of a pool is a pure function of (seed, tensor id, flat element
index), so the host can materialise any page it wants to check while the
device fills a pool of tens of GB in place, and both see the same bytes.

Value recipe: a 32-bit avalanche hash of the element index; the four bytes of
the hash are summed (Irwin-Hall, n=4), centred and scaled to unit variance,
then rounded to bfloat16.  The result is a symmetric bell-shaped variate with
variance 1 and support about +-3.45, standing in for N(0,1) cache contents.
"""
import numpy as np

from .bf16 import f32_to_bf16_bits

_M32 = 0xFFFFFFFF
# 4 independent uniform bytes: mean 4*127.5 = 510, variance 4*(256^2-1)/12 = 21845
_CENTRE = 510
_INV_SIGMA = np.float32(1.0 / np.sqrt(21845.0))

K_POOL_ID = 1
V_POOL_ID = 2


def _mix_np(lo: np.ndarray, hi: np.ndarray, seed: int, tensor_id: int) -> np.ndarray:
    m = np.uint64(_M32)
    x = (lo * np.uint64(0x9E3779B1) + hi * np.uint64(0x85EBCA77)
         + np.uint64((seed * 0xC2B2AE3D + tensor_id * 0x27D4EB2F + 0x165667B1) & _M32)) & m
    x ^= x >> np.uint64(16)
    x = (x * np.uint64(0x85EBCA6B)) & m
    x ^= x >> np.uint64(13)
    x = (x * np.uint64(0xC2B2AE35)) & m
    x ^= x >> np.uint64(16)
    return x


def pool_bits_np(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """bf16 bit patterns of pool elements [start, start+count) (flat index)."""
    idx = np.arange(start, start + count, dtype=np.uint64)
    x = _mix_np(idx & np.uint64(_M32), idx >> np.uint64(32), seed, tensor_id)
    s = ((x & np.uint64(255)) + ((x >> np.uint64(8)) & np.uint64(255))
         + ((x >> np.uint64(16)) & np.uint64(255)) + ((x >> np.uint64(24)) & np.uint64(255)))
    f = (s.astype(np.int64) - _CENTRE).astype(np.float32) * _INV_SIGMA
    return f32_to_bf16_bits(f)


def pool_fill_torch(pool, seed: int, tensor_id: int, chunk: int = 1 << 26) -> None:
    """Fill a contiguous torch.bfloat16 tensor in place with the same values
    pool_bits_np() yields, on whatever device the tensor lives on."""
    import torch

    flat = pool.view(-1)
    n = flat.numel()
    dev = flat.device
    const = (seed * 0xC2B2AE3D + tensor_id * 0x27D4EB2F + 0x165667B1) & _M32
    inv_sigma = float(_INV_SIGMA)
    for start in range(0, n, chunk):
        cnt = min(chunk, n - start)
        idx = torch.arange(start, start + cnt, dtype=torch.int64, device=dev)
        lo = idx & _M32
        hi = idx >> 32
        x = (lo * 0x9E3779B1 + hi * 0x85EBCA77 + const) & _M32
        x = x ^ (x >> 16)
        x = (x * 0x85EBCA6B) & _M32
        x = x ^ (x >> 13)
        x = (x * 0xC2B2AE35) & _M32
        x = x ^ (x >> 16)
        s = (x & 255) + ((x >> 8) & 255) + ((x >> 16) & 255) + ((x >> 24) & 255)
        f = (s - _CENTRE).to(torch.float32) * torch.tensor(inv_sigma, dtype=torch.float32, device=dev)
        flat[start:start + cnt] = f.to(torch.bfloat16)
