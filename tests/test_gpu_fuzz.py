"""Seeded sweep over small random configurations: shapes, ragged lengths, chunk offsets, budget modes and
schedule / kernel flags, each compared with the CPU oracle through the C ABI (same tolerances as elsewhere)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_09508_b200 as ei
import synth
from util import bf16_bits_to_f64, lists_of, to_bits, to_dev

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def draw(seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    if seed >= 100:                                              # a second family of seeds: head_dim 256
        d = 256
    L_B = int(rng.choice([64, 128]))
    L_S = int(rng.choice([m for m in (128, 256, 512) if m % L_B == 0]))
    if seed >= 200:                                              # a third family: the shape of the tile-pair kernels
        d, L_B, L_S = 128, 128, (256, 512)[seed % 2]
    Hkv = int(rng.choice([1, 2, 3]))
    G = int(rng.choice([1, 2, 4, 7]))
    n_blocks = int(rng.integers(3, 40))
    N = n_blocks * L_B - int(rng.integers(0, L_B))               # usually not a multiple of anything
    chunk = bool(rng.integers(0, 2))
    P = int(rng.integers(1, max(2, N // L_B))) * L_B if chunk and N > 2 * L_B else 0
    mode = str(rng.choice(["total", "base"]))
    f = float(rng.choice([0.2, 0.4, 0.7, 1.0]))
    flags = 0
    if rng.integers(0, 2):
        flags |= ei.FLAG_GROUP_SHARED
    flags |= int(rng.choice([0, ei.FLAG_PLAN_FUSED, ei.FLAG_PLAN_STAGED]))
    flags |= int(rng.choice([0, ei.FLAG_ATTN_PERSISTENT, ei.FLAG_ATTN_SINGLE_TILE, ei.FLAG_ATTN_PAIR_8WARP, ei.FLAG_ATTN_PER_CTA]))
    if seed % 5 == 3:                                            # every fifth configuration: all probabilities evaluated
        flags |= ei.FLAG_ATTN_NO_SKIP
    if seed >= 200:                                              # the three-buffer kernel where the shape allows it
        flags |= ei.FLAG_ATTN_TRI
    return dict(H=Hkv * G, Hkv=Hkv, d=d, N=N, P=P, L_S=L_S, L_B=L_B, mode=mode, f=f, flags=flags, seed=seed)


@pytest.mark.parametrize("seed", list(range(28)) + list(range(100, 112)) + list(range(200, 212)))
def test_random_configuration(seed):
    c = draw(seed)
    H, Hkv, d, N, P, L_S, L_B = (c[k] for k in ("H", "Hkv", "d", "N", "P", "L_S", "L_B"))
    Nq = N - P
    q, k, v = synth.generate_plain(H, Hkv, N, d, seed=500 + seed)   # unit scale: the absolute output tolerance assumes it
    qc = np.ascontiguousarray(q[:, P:])
    group = bool(c["flags"] & ei.FLAG_GROUP_SHARED)
    kw = dict(fraction=c["f"]) if c["mode"] == "total" else dict(base_tokens=float(2 * L_B + 37))
    p = ei.params_default(H, Hkv, d, N, L_S, L_B, c["f"] if c["mode"] == "total" else 0.0)
    if c["mode"] == "base":
        p.base_budget_tokens = float(2 * L_B + 37)
    if P:
        p.q_len = Nq
        p.q_stride_head = p.o_stride_head = Nq * d
    p.flags = c["flags"]
    try:
        op = oracle.plan(qc, k, L_S, L_B, group_shared=group, **kw)
    except ValueError:                                   # total below the forced minimum: the library must refuse too
        with pytest.raises(ei.EiError):
            ei.Plan(p)
        return
    pl = ei.Plan(p)
    qd, kd, vd = to_dev(qc), to_dev(k), to_dev(v)
    out = torch.full((H, Nq, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    pl.plan(qd, kd)
    pl.sparse_prefill(qd, kd, vd, out)
    res = pl.results()
    assert pl.status() == 0, c
    C_S = -(-Nq // L_S)
    heads = Hkv if group else H
    # stage 1: entropies and scores of the query heads
    e = res["entropy"].astype(np.float64)
    ref_e = op.head_entropy64 if group else op.entropy64
    assert (np.abs(e - ref_e) <= 1e-3 * np.abs(ref_e) + 1e-7).all(), c
    # stages 2-3 on the GPU's own entropy table
    tab = res["group_entropy"] if group else res["entropy"]
    want = oracle.plan(qc, k, L_S, L_B, group_shared=group, entropy_override=tab, **kw)
    np.testing.assert_array_equal(res["k"], want.k, err_msg=str(c))
    got_l = lists_of(res["offsets"], res["idx"], heads * C_S)
    ref_l = lists_of(want.offsets, want.idx, heads * C_S)
    bad = [cc for cc in range(heads * C_S) if not np.array_equal(got_l[cc], ref_l[cc]) and want.gap[cc] >= 1e-4]
    assert not bad, (c, bad[:4])
    # stage 4 on the GPU's own lists
    off, idx = res["offsets"].astype(np.int64), res["idx"]
    if group:
        off, idx = oracle.expand_group_lists(off, idx, Hkv, H // Hkv, C_S)
    ref = oracle.sparse_attention(qc, k, v, L_S, L_B, off, idx).reshape(H, C_S * L_S, d)[:, :Nq]
    got = bf16_bits_to_f64(to_bits(out))
    assert np.isfinite(got).all(), c
    err = np.abs(got - ref)
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (c, err.max(), err.mean())
