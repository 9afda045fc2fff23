"""A layer's heads sharded over several plans by KV group (ei_plan_observe, ei_stage_multipliers, gathered tables,
ei_stage_apportion, ei_stage_select): the shards' rows must be the rows of one plan over all heads, bit for bit.
The shards run one after another on one GPU; the gathered table is assembled in place of the all-gather."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2606_09508_b200 as ei
import synth
from util import lists_of, to_bits, to_dev

pytestmark = pytest.mark.gpu

WL = synth.Workload("shard", 8, 4, 128, 4096, 512, 128, 0.30, 0.5, 2, 3, seed=91)


def _total_all(wl, fraction):
    SC = sum(min(wl.r * (i + 1), wl.C_B) for i in range(wl.C_S))
    return int(math.floor(fraction * float(wl.H) * float(SC) + 0.5))


def _full(wl, q, k, v, fraction=None, base_tokens=None, flags=0):
    p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, fraction or 0.0)
    if base_tokens:
        p.base_budget_tokens = base_tokens
    p.flags = flags
    pl = ei.Plan(p)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    out = torch.empty((wl.H, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
    pl.plan(qd, kd)
    pl.sparse_prefill(qd, kd, vd, out)
    assert pl.status() == 0
    return pl.results(), to_bits(out)


@pytest.mark.parametrize("world", [1, 2, 4])
@pytest.mark.parametrize("mode", ["total", "base"])
def test_shards_equal_the_unsharded_plan(world, mode):
    wl = WL
    q, k, v, _ = synth.generate(wl)
    kw = dict(fraction=wl.fraction) if mode == "total" else dict(base_tokens=640.0)
    ref, ref_out = _full(wl, q, k, v, **kw)
    G, gper = wl.H // wl.Hkv, wl.Hkv // world
    T_all = _total_all(wl, wl.fraction) if mode == "total" else 0
    m_all = torch.zeros((wl.H, wl.C_S), dtype=torch.int32, device="cuda")
    plans, devs = [], []
    for p_ in range(world):
        g0, g1 = p_ * gper, (p_ + 1) * gper
        h0, h1 = g0 * G, g1 * G
        pr = ei.params_default(h1 - h0, g1 - g0, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction if mode == "total" else 0.0)
        if mode == "base":
            pr.base_budget_tokens = 640.0
        pr.flags = ei.FLAG_HEAD_SHARD
        pl = ei.Plan(pr)
        qd, kd, vd = to_dev(q[h0:h1]), to_dev(k[g0:g1]), to_dev(v[g0:g1])
        pl.observe(qd, kd)
        pl.stage_multipliers(out=m_all[h0:h1])          # this shard's rows of the gathered table
        plans.append((pl, h0, h1))
        devs.append((qd, kd, vd))
    torch.cuda.synchronize()
    for (pl, h0, h1), (qd, kd, vd) in zip(plans, devs):
        pl.stage_apportion(m_all, wl.H, h0, T_all if mode == "total" else 1)
        pl.stage_select()
        out = torch.empty((h1 - h0, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
        pl.sparse_prefill(qd, kd, vd, out)
        res = pl.results()
        assert pl.status() == 0
        cells = (h1 - h0) * wl.C_S
        lo = int(ref["offsets"][h0 * wl.C_S])
        np.testing.assert_array_equal(res["rigid"], ref["rigid"][h0:h1])
        np.testing.assert_array_equal(res["k"], ref["k"][h0:h1])
        np.testing.assert_array_equal(res["offsets"], ref["offsets"][h0 * wl.C_S:h0 * wl.C_S + cells + 1] - lo)
        n = int(res["offsets"][-1])
        np.testing.assert_array_equal(res["idx"][:n], ref["idx"][lo:lo + n])
        np.testing.assert_array_equal(to_bits(out), ref_out[h0:h1])
        if mode == "total":                              # b* and the leftover are the layer's
            np.testing.assert_array_equal(res["stats"][2:4], ref["stats"][2:4])
            assert int(res["stats"][0]) == n
    if mode == "total":
        # the gathered table is the oracle's multiplier table of the GPU's own entropies, and its apportionment
        # of the layer's total gives the counts the shards ended up with
        ent = np.concatenate([pl.read("ENTROPY").reshape(h1 - h0, wl.C_S) for pl, h0, h1 in plans])
        _, m = oracle.multipliers(ent)
        np.testing.assert_array_equal(m_all.cpu().numpy(), np.floor(m * 4096.0 + 0.5).astype(np.int32))
        k_or, _ = oracle.budgets_total(m, wl.r, T_all)
        np.testing.assert_array_equal(np.concatenate([pl.read("BUDGET").reshape(h1 - h0, wl.C_S) for pl, h0, h1 in plans]), k_or)


def test_shard_errors():
    wl = WL
    q, k, v, _ = synth.generate(wl)
    m_all = torch.full((wl.H, wl.C_S), 4096, dtype=torch.int32, device="cuda")
    pr = ei.params_default(4, 2, wl.d, wl.N, wl.L_S, wl.L_B, 0.30)
    pl = ei.Plan(pr)                                     # no EI_FLAG_HEAD_SHARD: index buffer for its own share only
    T_all = _total_all(wl, 0.9)
    with pytest.raises(ei.EiError) as e:
        pl.stage_apportion(m_all, wl.H, 0, T_all)
    assert e.value.code == ei.STATUS["PLAN_MISMATCH"]
    pr.flags = ei.FLAG_HEAD_SHARD
    pl = ei.Plan(pr)
    with pytest.raises(ei.EiError) as e:
        pl.stage_apportion(m_all, wl.H, 0, 3)            # below the forced diagonal blocks
    assert e.value.code == ei.STATUS["BUDGET_INFEASIBLE"]
    with pytest.raises(ei.EiError) as e:
        pl.stage_apportion(m_all, wl.H, 6, T_all)        # my 4 heads do not fit behind head 6 of 8
    assert e.value.code == ei.STATUS["INVALID_ARG"]
