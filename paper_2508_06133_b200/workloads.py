"""Seeded synthetic request backlogs (inputs only; none of the scheduling method lives here).

Every instance is a pair of int32 arrays (s, o) -- prefill and decode lengths of n requests that
are all present at t = 0 (Section 2.1, "Request Arrivals") -- plus a KV budget M.  The shapes follow
the paper's experiments (Section 7, "Dataset Overview"): a bimodal mixture of many short chats and a
minority of long-prompt summarisation requests, served in the overloaded regime n*L/M >> 1.  The
paper's own token-length samples come from two public datasets that are not shipped here, so these
draws stand in for them.

Random numbers come from one counter-based generator, so any element can be recomputed on its own:

    u64(seed, stream, k) = splitmix64_finaliser(seed * C1 + stream * C2 + k * C3)     (mod 2^64)

Uniform doubles take the top 53 bits; normals use Box-Muller in float64; integers are rounded half
away from zero and clipped.  The same arrays are handed to the CPU checker and to the GPU library.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_C1 = np.uint64(0x9E3779B97F4A7C15)
_C2 = np.uint64(0xD1B54A32D192ED03)
_C3 = np.uint64(0x8CB92BA72F3D8DD7)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.uint64, copy=True)
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def u64(seed: int, stream: int, k: np.ndarray) -> np.ndarray:
    """Counter-based 64-bit words for counters ``k`` of one (seed, stream)."""
    with np.errstate(over="ignore"):
        base = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _C1 + np.uint64(stream) * _C2
        return _mix(base + np.asarray(k, dtype=np.uint64) * _C3)


def uniform01(seed: int, stream: int, k: np.ndarray) -> np.ndarray:
    """Doubles in [0, 1) from the top 53 bits."""
    return (u64(seed, stream, k) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def uniform_int(seed: int, stream: int, k: np.ndarray, lo: int, hi: int) -> np.ndarray:
    """Integers in [lo, hi] (inclusive)."""
    span = np.uint64(hi - lo + 1)
    return (u64(seed, stream, k) % span).astype(np.int64) + lo


def normal(seed: int, stream: int, k: np.ndarray) -> np.ndarray:
    """Standard normals by Box-Muller; streams ``stream`` and ``stream + 1`` are consumed."""
    u1 = 1.0 - uniform01(seed, stream, k)          # (0, 1]
    u2 = uniform01(seed, stream + 1, k)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def lognormal_int(seed: int, stream: int, k: np.ndarray, mu: float, sigma: float,
                  lo: int, hi: int) -> np.ndarray:
    x = np.exp(mu + sigma * normal(seed, stream, k))
    r = np.floor(x + 0.5)                           # x > 0: round half away from zero
    return np.clip(r, lo, hi).astype(np.int64)


@dataclass(frozen=True)
class Instance:
    name: str
    s: np.ndarray          # int32 [n]   prefill lengths
    o: np.ndarray          # int32 [n]   decode lengths
    M: int                 # KV budget in tokens

    @property
    def n(self) -> int:
        return int(self.s.shape[0])

    def checksum(self) -> int:
        """FNV-1a over the little-endian bytes of s, o and M; logged so both sides see one input."""
        h = 0xCBF29CE484222325
        data = self.s.astype("<i4").tobytes() + self.o.astype("<i4").tobytes() + int(self.M).to_bytes(8, "little")
        arr = np.frombuffer(data, dtype=np.uint8)
        for chunk in np.array_split(arr, max(1, arr.size // 4096)):
            for b in chunk.tolist():
                h = ((h ^ b) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
        return h


def uniform_backlog(n: int, seed: int, lo: int, hi: int, M: int, name: str = "uniform") -> Instance:
    k = np.arange(n)
    s = uniform_int(seed, 0, k, lo, hi)
    o = uniform_int(seed, 1, k, lo, hi)
    return Instance(name, s.astype(np.int32), o.astype(np.int32), M)


def mixed_backlog(n: int, seed: int, M: int, *, frac_long: float = 0.2,
                  chat_s=(5.5, 0.8, 16, 2048), chat_o=(5.0, 0.9, 8, 1024),
                  doc_s=(4096, 16384), doc_o=(128, 512), name: str = "mixed") -> Instance:
    """Short chats (log-normal lengths) mixed with long-document requests (uniform lengths)."""
    k = np.arange(n)
    is_doc = uniform01(seed, 0, k) < frac_long
    cs = lognormal_int(seed, 1, k, *chat_s)
    co = lognormal_int(seed, 3, k, *chat_o)
    ds = uniform_int(seed, 5, k, *doc_s)
    do = uniform_int(seed, 6, k, *doc_o)
    s = np.where(is_doc, ds, cs)
    o = np.where(is_doc, do, co)
    inst = Instance(name, s.astype(np.int32), o.astype(np.int32), M)
    assert int((inst.s.astype(np.int64) + inst.o).max()) <= M
    return inst


def tiny(seed: int = 0) -> Instance:
    """n = 16, s and o uniform on 1..32, M = 256."""
    return uniform_backlog(16, seed, 1, 32, 256, name="tiny_n16")


def mixed_1k(seed: int = 1) -> Instance:
    return mixed_backlog(1000, seed, 65536, name="mixed_n1000")


def mixed_10k(seed: int = 2) -> Instance:
    """Headline backlog: n = 10,000, M = 262,144."""
    return mixed_backlog(10000, seed, 262144, name="mixed_n10000")


def policy_sweep(num_instances: int = 4096, n_each: int = 256, first_seed: int = 3, M: int = 32768):
    """``num_instances`` independent backlogs; returns (s[B, n], o[B, n], M)."""
    s = np.empty((num_instances, n_each), dtype=np.int32)
    o = np.empty((num_instances, n_each), dtype=np.int32)
    for b in range(num_instances):
        inst = mixed_backlog(n_each, first_seed + b, M, name="sweep")
        s[b], o[b] = inst.s, inst.o
    return s, o, M


def heavy_100k(seed: int = 5) -> Instance:
    """n = 100,000 with a heavier tail: 70 % chats, 30 % long documents, M = 4,194,304."""
    return mixed_backlog(100000, seed, 4194304, frac_long=0.3,
                         chat_s=(6.0, 1.0, 16, 8192), chat_o=(5.5, 1.0, 8, 4096),
                         doc_s=(8192, 32768), doc_o=(256, 1024), name="heavy_n100000")


def paper_scale(seed: int = 7, n: int = 2000) -> Instance:
    """The paper's own scale (Section 7: n = 2000, M = 16,492) with log-normals matched to the
    printed medians/means of the two datasets; documents clipped so that s + o <= M."""
    return mixed_backlog(n, seed, 16492, chat_s=(2.48, 1.58, 1, 4096), chat_o=(3.76, 1.17, 1, 2048),
                         doc_s=(500, 4800), doc_o=(30, 560), name="paper_scale_n%d" % n)


def random_permutations(n: int, count: int, seed: int) -> np.ndarray:
    """``count`` permutations of 0..n-1 (int32 [count, n]) by sorting counter-based keys."""
    out = np.empty((count, n), dtype=np.int32)
    k = np.arange(n)
    for c in range(count):
        out[c] = np.argsort(u64(seed, 100 + c, k), kind="stable").astype(np.int32)
    return out


@dataclass(frozen=True)
class OnlineInstance:
    name: str
    a: np.ndarray          # int32 [n]   arrival times, non-decreasing
    s: np.ndarray          # int32 [n]
    o: np.ndarray          # int32 [n]
    M: int

    @property
    def n(self) -> int:
        return int(self.s.shape[0])


def online_poisson(lam: float, horizon: int = 4000, seed: int = 11, M: int = 16492) -> OnlineInstance:
    """Poisson arrivals of rate ``lam`` per iteration over ``horizon`` iterations (Section 7, online
    experiment): exponential gaps from the counter-based generator, arrival time = floor of the
    running sum, arrivals at or after ``horizon`` dropped; lengths as in ``paper_scale``."""
    kmax = int(lam * horizon * 1.5 + 64)
    k = np.arange(kmax)
    gaps = -np.log(1.0 - uniform01(seed, 40, k)) / lam
    times = np.floor(np.cumsum(gaps)).astype(np.int64)
    n = int(np.searchsorted(times, horizon, side="left"))
    n = max(n, 1)
    base = paper_scale(seed=seed, n=kmax)
    return OnlineInstance("online_lam%.2f_seed%d" % (lam, seed), times[:n].astype(np.int32),
                          base.s[:n].copy(), base.o[:n].copy(), M)


def memory_bound_rate(s: np.ndarray, o: np.ndarray, M: int) -> float:
    """Arrival rate at which the mean KV-memory demand per iteration equals M: a request holds
    s + j tokens in its j-th round, so it needs sum_j (s + j) token-rounds."""
    s = s.astype(np.float64)
    o = o.astype(np.float64)
    return float(M / np.mean(o * s + o * (o + 1) / 2))
