"""Seeded synthetic Q/K/V for the EntropyInfer prefill path.

This module only makes inputs: it holds none of the method's arithmetic and is the
one piece shared by the CPU oracle's tests and the CUDA path's tests / benchmark.

The paper evaluates on real-model activations of long documents; those are not
available, so each workload below takes the attention shape of the named model
and plants the two head regimes the paper describes (Motivation 1):

* Rigid heads  -- an attention-sink key at position 0 that every query of the
  head is aligned with, so the pooled observation attention is one-hot.
* Dynamic heads -- per query segment, a few random earlier key blocks
  ("needles") that the segment's queries are aligned with at a random strength,
  so the observation entropy moves from segment to segment.

Recipe (all draws from Philox streams keyed by (seed, tensor, head)):
 1. Q[h,t,:], K[g,t,:], V[g,t,:] ~ N(0,1) i.i.d.
 2. round(rho*H) query heads, chosen by a seeded permutation, are Rigid.
 3. Needles: per KV head g and key block j a direction w[g,j] = Rademacher/sqrt(d);
    every key of block j gets  + d^(1/4) * w[g,j].  For every Dynamic head and
    every segment i >= 1, n distinct blocks j < r*i are drawn, a ~ U[0,6] once
    per segment, and every query of the segment gets + a * d^(1/4) * w[g,j] for
    each drawn j (a logit gain of a on those blocks).
 4. Sink: per KV head g that serves a Rigid head, u[g] in {+-1}^d;
    K[g,0,:] = 8*u[g]; every query of a Rigid head gets + 8*u[g]
    (a per-coordinate amplitude, so that min/max pooling still sees it).
Values are rounded once to bf16 (round-to-nearest-even); both sides read the same bits.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    H: int
    Hkv: int
    d: int
    N: int
    L_S: int
    L_B: int
    fraction: float          # budget as a fraction of causal blocks (TOTAL mode)
    rigid_fraction: float    # rho; < 0 means "draw U[0.2, 0.8] from the seed"
    needles_lo: int
    needles_hi: int          # inclusive; needle count per segment ~ U{lo..hi}
    seed: int = 0

    @property
    def r(self) -> int:
        return self.L_S // self.L_B

    @property
    def C_S(self) -> int:
        return self.N // self.L_S

    @property
    def C_B(self) -> int:
        return self.N // self.L_B

    @property
    def G(self) -> int:
        return self.H // self.Hkv

    @property
    def sum_causal(self) -> int:
        return self.r * self.C_S * (self.C_S + 1) // 2


# The five benchmark workloads (tiny oracle check; Llama-3-8B at 32k and 128k;
# Qwen2.5-7B at 64k; Llama-3.1-70B-shaped sweep base at 128k, 5 %).
WORKLOADS = {
    "tiny": Workload("tiny", 8, 2, 64, 2048, 128, 64, 0.25, 0.5, 2, 2, seed=1000),
    "llama3_8b_32k": Workload("llama3_8b_32k", 32, 8, 128, 32768, 512, 128, 0.10, 0.5, 4, 4, seed=2000),
    "llama3_8b_128k": Workload("llama3_8b_128k", 32, 8, 128, 131072, 1024, 128, 0.05, 0.6, 2, 16, seed=3000),
    "qwen25_7b_64k": Workload("qwen25_7b_64k", 28, 4, 128, 65536, 512, 128, 0.08, -1.0, 2, 2, seed=4000),
    "llama31_70b_128k": Workload("llama31_70b_128k", 64, 8, 128, 131072, 1024, 128, 0.05, 0.5, 2, 2, seed=5000),
}


def with_(w: Workload, **kw) -> Workload:
    return replace(w, **kw)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (uint16). No NaNs expected."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    u = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, tensor: int, head: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) | tensor, (head << 16) | sub]))


_T_Q, _T_K, _T_V, _T_META, _T_NEEDLE, _T_W = 1, 2, 3, 4, 5, 6


@dataclass
class Structure:
    """The planted structure of one workload instance (inputs' ground truth)."""
    rigid: np.ndarray        # [H] bool, planted class
    sink_u: np.ndarray       # [Hkv, d] float32 in {+-1} (zero rows: no sink on that KV head)
    w: np.ndarray            # [Hkv, C_B, d] float32 needle directions (unit norm)
    rho: float


def structure(wl: Workload) -> Structure:
    meta = _rng(wl.seed, _T_META, 0)
    rho = wl.rigid_fraction if wl.rigid_fraction >= 0 else float(meta.uniform(0.2, 0.8))
    perm = meta.permutation(wl.H)
    rigid = np.zeros(wl.H, bool)
    rigid[perm[: int(round(rho * wl.H))]] = True
    sink_u = np.zeros((wl.Hkv, wl.d), np.float32)
    for g in range(wl.Hkv):
        u = _rng(wl.seed, _T_META, 1 + g).integers(0, 2, wl.d).astype(np.float32) * 2 - 1
        if rigid[g * wl.G:(g + 1) * wl.G].any():
            sink_u[g] = u
    w = np.empty((wl.Hkv, wl.C_B, wl.d), np.float32)
    for g in range(wl.Hkv):
        w[g] = (_rng(wl.seed, _T_W, g).integers(0, 2, (wl.C_B, wl.d)).astype(np.float32) * 2 - 1) \
            / np.float32(np.sqrt(wl.d))
    return Structure(rigid, sink_u, w, rho)


def gen_k_head(wl: Workload, st: Structure, g: int) -> np.ndarray:
    """K[g] as bf16 bits [N, d]."""
    k = _rng(wl.seed, _T_K, g).standard_normal((wl.N, wl.d), dtype=np.float32)
    amp = np.float32(wl.d ** 0.25)
    k.reshape(wl.C_B, wl.L_B, wl.d)[...] += amp * st.w[g][:, None, :]
    if st.sink_u[g].any():
        k[0, :] = 8.0 * st.sink_u[g]
    return f32_to_bf16_bits(k)


def gen_v_head(wl: Workload, g: int) -> np.ndarray:
    return f32_to_bf16_bits(_rng(wl.seed, _T_V, g).standard_normal((wl.N, wl.d), dtype=np.float32))


def needle_plan(wl: Workload, st: Structure, h: int):
    """For a Dynamic head: per segment i >= 1 the drawn blocks and strength."""
    rng = _rng(wl.seed, _T_NEEDLE, h)
    out = []
    for i in range(wl.C_S):
        ncand = wl.r * i
        n = int(rng.integers(wl.needles_lo, wl.needles_hi + 1))
        a = float(rng.uniform(0.0, 6.0))
        if ncand == 0:
            out.append((np.zeros(0, np.int64), 0.0))
            continue
        n = min(n, ncand)
        blocks = rng.choice(ncand, size=n, replace=False)
        out.append((np.sort(blocks), a))
    return out


def gen_q_head(wl: Workload, st: Structure, h: int) -> np.ndarray:
    """Q[h] as bf16 bits [N, d]."""
    g = h // wl.G
    q = _rng(wl.seed, _T_Q, h).standard_normal((wl.N, wl.d), dtype=np.float32)
    if st.rigid[h]:
        q += 8.0 * st.sink_u[g][None, :]
    else:
        amp = np.float32(wl.d ** 0.25)
        qs = q.reshape(wl.C_S, wl.L_S, wl.d)
        for i, (blocks, a) in enumerate(needle_plan(wl, st, h)):
            if len(blocks):
                qs[i] += np.float32(a) * amp * st.w[g][blocks].sum(axis=0)[None, :]
    return f32_to_bf16_bits(q)


def _workers() -> int:
    return max(1, min(16, os.cpu_count() or 1))


def generate(wl: Workload):
    """-> (q [H,N,d], k [Hkv,N,d], v [Hkv,N,d]) uint16 bf16 bits, and the Structure.

    Every head draws from a stream of its own, so the heads are generated by a pool of threads (numpy releases
    the interpreter lock while it draws); the result does not depend on how many threads there are."""
    st = structure(wl)
    q = np.empty((wl.H, wl.N, wl.d), np.uint16)
    k = np.empty((wl.Hkv, wl.N, wl.d), np.uint16)
    v = np.empty((wl.Hkv, wl.N, wl.d), np.uint16)

    def kv(g):
        k[g] = gen_k_head(wl, st, g)
        v[g] = gen_v_head(wl, g)

    def qh(h):
        q[h] = gen_q_head(wl, st, h)

    with ThreadPoolExecutor(_workers()) as pool:
        list(pool.map(kv, range(wl.Hkv)))
        list(pool.map(qh, range(wl.H)))
    return q, k, v, st


def generate_plain(H: int, Hkv: int, N: int, d: int, seed: int, scale: float = 1.0):
    """Structure-free N(0, scale^2) Q/K/V (bf16 bits) for exercising diffuse softmax rows."""
    def t(tensor, heads):
        out = np.empty((heads, N, d), np.uint16)

        def one(h):
            x = _rng(seed, tensor, h).standard_normal((N, d), dtype=np.float32)
            out[h] = f32_to_bf16_bits(x * np.float32(scale))
        with ThreadPoolExecutor(_workers()) as pool:
            list(pool.map(one, range(heads)))
        return out
    return t(_T_Q, H), t(_T_K, Hkv), t(_T_V, Hkv)


def rope_tables(N: int, d: int, base: float = 500000.0, pos0: int = 0):
    """cos / sin tables [N, d/2] float32 of the rotary angles pos * base^(-2j/d), positions pos0 .. pos0+N-1
    (base 500000: the Llama-3 setting).  Inputs of the producer step, handed to both sides."""
    j = np.arange(d // 2, dtype=np.float64)
    inv_freq = base ** (-2.0 * j / d)
    ang = (pos0 + np.arange(N, dtype=np.float64))[:, None] * inv_freq[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
