"""Seeded synthetic CTB batches (input generation only, no attention or paging arithmetic).

Five workloads shaped like the paper's multi-turn text and multimodal agent
rollouts (trajectory statistics: paper Appendix C, Table 4), as stand-ins for
its datasets, which are not needed: only shapes and length mixes matter here.
Both the CUDA library's tests and the CPU oracle's tests draw their inputs
from this module, as identical bf16 bit patterns (numpy uint16).

A workload is a list of tasks, each with a preserved prefix p (the KV state a
paused task keeps) and n_new tokens appended when it resumes (1 for a decode
row).  Lengths come from numpy.random.default_rng(1000 + k) for workload k;
values come from a generator keyed by (seed, task id, stream).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

K = 1024  # "1k" tokens


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, sigma: float = 1.0) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if sigma != 1.0:
        x *= np.float32(sigma)
    return f32_to_bf16_bits(x)


@dataclass
class Workload:
    name: str
    index: int                 # 1..5
    seed: int
    Hq: int
    Hkv: int
    D: int
    S: int
    scale: float
    task: np.ndarray           # [B] task ids, in batch order
    prefix: np.ndarray         # [B] preserved context p
    n_new: np.ndarray          # [B] appended tokens (q_len); 1 = decode row
    n_image: np.ndarray        # [B] how many of the appended tokens are image tokens (first in the chunk)
    image_sigma: float = 1.5
    num_pages: int = 0
    max_tasks: int = 0
    max_pages_per_task: int = 0
    free_order: np.ndarray = field(default=None, repr=False)

    @property
    def B(self) -> int:
        return int(self.task.shape[0])

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def ctx(self) -> np.ndarray:
        return self.prefix + self.n_new

    def rows(self):
        """[(task, q_len, ctx_len)] in batch order."""
        return [(int(t), int(n), int(p + n)) for t, p, n in zip(self.task, self.prefix, self.n_new)]

    def kv_bytes_per_token(self) -> int:
        return self.Hkv * self.D * 2 * 2

    def decode_kv_bytes(self) -> int:
        d = self.n_new == 1
        return int(self.kv_bytes_per_token() * int(self.ctx[d].sum()))

    def resume_pairs(self) -> int:
        r = self.n_new > 1
        n, p = self.n_new[r].astype(np.int64), self.prefix[r].astype(np.int64)
        return int((n * p + n * (n + 1) // 2).sum())

    def resume_flops(self) -> int:
        return 4 * self.D * self.Hq * self.resume_pairs()

    def live_pages(self) -> int:
        return int(((self.ctx + self.S - 1) // self.S).sum())

    # ---- values ------------------------------------------------------------
    def _rng(self, task: int, stream: int) -> np.random.Generator:
        return np.random.default_rng([self.seed, int(task), stream])

    def task_kv(self, b: int):
        """K and V bits [p + n_new, Hkv, D] of batch row b's task (prefix then appended chunk)."""
        p, n, ni = int(self.prefix[b]), int(self.n_new[b]), int(self.n_image[b])
        t = int(self.task[b])
        L = p + n
        k = normal_bf16(self._rng(t, 0), (L, self.Hkv, self.D))
        v = normal_bf16(self._rng(t, 1), (L, self.Hkv, self.D))
        if ni > 0:
            k[p:p + ni] = normal_bf16(self._rng(t, 3), (ni, self.Hkv, self.D), self.image_sigma)
            v[p:p + ni] = normal_bf16(self._rng(t, 4), (ni, self.Hkv, self.D), self.image_sigma)
        return k, v

    def task_q_full(self, b: int):
        """Q bits for EVERY position of the task [p + n_new, Hq, D]; the row's queries are the last n_new."""
        t = int(self.task[b])
        L = int(self.prefix[b] + self.n_new[b])
        return normal_bf16(self._rng(t, 2), (L, self.Hq, self.D))

    def task_q(self, b: int):
        return self.task_q_full(b)[int(self.prefix[b]):]


def _lognormal_lengths(rng, n, median, lo, hi, sigma=1.0):
    x = median * np.exp(sigma * rng.standard_normal(n))
    return np.clip(np.rint(x), lo, hi).astype(np.int64)


def _pareto_lengths(rng, n, xm, alpha, hi):
    u = 1.0 - rng.random(n)          # (0, 1]
    x = xm * u ** (-1.0 / alpha)
    return np.clip(np.rint(x), xm, hi).astype(np.int64)


def make_workload(index: int, seed: int | None = None, n_tasks: int | None = None, len_div: int = 1,
                  pool_factor: float | None = None) -> Workload:
    """Workload `index` (1..5).  n_tasks / len_div shrink it for quick parity
    cases: fewer tasks (the decode/resume mix is kept), and every length bound
    divided by len_div.  pool_factor = pool pages / live pages."""
    if seed is None:
        seed = 1000 + index
    rng = np.random.default_rng(seed)
    dv = max(1, int(len_div))

    def sc(x):  # scaled length bound
        return max(1, int(x) // dv)

    image = None
    if index == 1:
        name, (Hq, Hkv, D, S) = "tiny CTB step", (8, 2, 64, 16)
        B = n_tasks or 4
        n_res = B // 2
        prefix = rng.integers(sc(200), sc(600) + 1, size=B)
        n_new = np.concatenate([np.ones(B - n_res, np.int64), rng.integers(sc(32), sc(64) + 1, size=n_res)])
        pf = pool_factor or 2.0
    elif index == 2:
        name, (Hq, Hkv, D, S) = "decode-only continuous batch", (28, 4, 128, 16)
        B = n_tasks or 64
        prefix = _lognormal_lengths(rng, B, sc(4 * K), sc(1 * K), sc(32 * K))
        prefix[0] = sc(32 * K)  # always exercise the longest path
        n_new = np.ones(B, np.int64)
        pf = pool_factor or 4.0
    elif index == 3:
        name, (Hq, Hkv, D, S) = "mixed multi-turn text resume batch", (28, 4, 128, 16)
        B = n_tasks or 128
        n_res = B // 4
        prefix = _lognormal_lengths(rng, B, sc(8 * K), sc(2 * K), sc(32 * K))
        prefix[0] = sc(32 * K)
        n_new = np.concatenate([np.ones(B - n_res, np.int64), rng.integers(sc(200), sc(2000) + 1, size=n_res)])
        pf = pool_factor or 2.0
    elif index == 4:
        name, (Hq, Hkv, D, S) = "multimodal agent resume batch", (32, 8, 128, 16)
        B = n_tasks or 32
        prefix = _lognormal_lengths(rng, B, sc(16 * K), sc(4 * K), sc(64 * K))
        prefix[0] = sc(64 * K)
        image = rng.integers(sc(1000), sc(3000) + 1, size=B)
        text = rng.integers(sc(50), sc(200) + 1, size=B)
        n_new = image + text
        pf = pool_factor or 2.0
    elif index == 5:
        name, (Hq, Hkv, D, S) = "long-horizon stress batch", (28, 4, 128, 32)
        B = n_tasks or 256
        n_res = max(1, round(B * 26 / 256))
        prefix = _pareto_lengths(rng, B, sc(1 * K), 1.5, sc(128 * K))
        prefix[0] = sc(128 * K)
        n_new = np.concatenate([np.ones(B - n_res, np.int64), rng.integers(sc(500), sc(4000) + 1, size=n_res)])
        pf = pool_factor or 2.0
    else:
        raise ValueError("workload index must be 1..5")
    n_image = image if image is not None else np.zeros(B, np.int64)
    # resume rows were generated last; shuffle the batch order
    order = rng.permutation(B)
    prefix, n_new, n_image = prefix[order], n_new[order], n_image[order]
    task = np.arange(B, dtype=np.int64)
    w = Workload(name=name, index=index, seed=int(seed), Hq=Hq, Hkv=Hkv, D=D, S=S, scale=1.0 / math.sqrt(D),
                 task=task, prefix=prefix.astype(np.int64), n_new=n_new.astype(np.int64),
                 n_image=n_image.astype(np.int64))
    live = w.live_pages()
    w.num_pages = int(math.ceil(live * pf)) + 8
    w.max_tasks = B
    w.max_pages_per_task = int(((w.ctx + S - 1) // S).max()) + 1
    w.free_order = rng.permutation(w.num_pages).astype(np.int32)
    return w


def hashed_bf16_bits(task: int, start: int, count: int, Hkv: int, D: int, stream: int) -> np.ndarray:
    """Cheap reproducible bf16 filler [count, Hkv, D] for paused residents whose values are only
    checksummed: an integer hash of (task, position, head, d, stream) mapped to a bf16 in roughly
    [-2, 2).  Pure integer arithmetic, so any array library reproduces it bit for bit."""
    pos = np.arange(start, start + count, dtype=np.uint64)[:, None, None]
    h = np.arange(Hkv, dtype=np.uint64)[None, :, None]
    d = np.arange(D, dtype=np.uint64)[None, None, :]
    x = (pos * np.uint64(0x9E3779B1) + h * np.uint64(0x85EBCA77) + d * np.uint64(0xC2B2AE3D)
         + np.uint64(task) * np.uint64(0x27D4EB2F) + np.uint64(stream) * np.uint64(0x165667B1)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(15)
    x = (x * np.uint64(0x2C1B3C6D)) & np.uint64(0xFFFFFFFF)
    x ^= x >> np.uint64(12)
    # sign (1) | exponent in {125,126,127,128} (value magnitude 0.25..4) | 7 mantissa bits
    sign = (x & np.uint64(1)) << np.uint64(15)
    expo = (np.uint64(125) + ((x >> np.uint64(1)) & np.uint64(3))) << np.uint64(7)
    mant = (x >> np.uint64(3)) & np.uint64(0x7F)
    return (sign | expo | mant).astype(np.uint16)


def hashed_bf16_bits_torch(torch, task: int, start: int, count: int, Hkv: int, D: int, stream: int, device="cuda"):
    """The same filler as hashed_bf16_bits, produced on `device` with torch integer ops (int16 bit patterns)."""
    pos = torch.arange(start, start + count, dtype=torch.int64, device=device)[:, None, None]
    h = torch.arange(Hkv, dtype=torch.int64, device=device)[None, :, None]
    d = torch.arange(D, dtype=torch.int64, device=device)[None, None, :]
    x = (pos * 0x9E3779B1 + h * 0x85EBCA77 + d * 0xC2B2AE3D + int(task) * 0x27D4EB2F + int(stream) * 0x165667B1) & 0xFFFFFFFF
    x = x ^ (x >> 15)
    x = (x * 0x2C1B3C6D) & 0xFFFFFFFF
    x = x ^ (x >> 12)
    bits = ((x & 1) << 15) | ((125 + ((x >> 1) & 3)) << 7) | ((x >> 3) & 0x7F)
    return bits.to(torch.int32).to(torch.int16)   # two's-complement wrap keeps the 16 bit pattern
