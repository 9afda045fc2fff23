"""A device-side wait that runs out: reported through the plan's status word, the kernel returns, the plan and
the context stay usable.  No GPU is faulted, trapped or hung: the producer warp is told to leave one K/V load
out and the wait bound is shortened to 2^16 clocks, so the consumer's bounded wait simply expires."""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_09508_b200 as ei
import synth
from util import bf16_bits_to_f64, to_bits, to_dev

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_plan_stays_usable():
    H, Hkv, d, N, L_S, L_B = 2, 1, 128, 1024, 256, 128           # 8 tile pairs, lists of 2..8 blocks
    wl = synth.Workload("t", H, Hkv, d, N, L_S, L_B, 1.0, 0.0, 0, 0)
    q, k, v = synth.generate_plain(H, Hkv, N, d, seed=77)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    kc = np.array([[wl.r * (i + 1) for i in range(wl.C_S)] for _ in range(H)], np.int32)   # every causal block
    idx = np.concatenate([np.arange(c, dtype=np.int32) for c in kc.ravel()])
    offsets = np.concatenate([[0], np.cumsum(kc.ravel())]).astype(np.int64)
    pl = ei.Plan(ei.params_default(H, Hkv, d, N, L_S, L_B, 1.0))
    pl.set_lists(kc, idx)
    out = torch.full((H, N, d), float("nan"), dtype=torch.bfloat16, device="cuda")

    pl.debug_waits(wait_limit_log2=16, skip_ring_item=3)          # the V tile of every pair's second block never arrives
    pl.sparse_prefill(qd, kd, vd, out)
    assert pl.status() == ei.STATUS["DEVICE_TIMEOUT"]            # the call returned, with the failure on record
    assert pl.status() == 0                                        # reading it cleared it

    pl.debug_waits(0, -1)                                          # as before: the same plan, the same context
    out.fill_(float("nan"))
    pl.sparse_prefill(qd, kd, vd, out)
    assert pl.status() == 0
    got = bf16_bits_to_f64(to_bits(out))
    want = oracle.sparse_attention(q, k, v, L_S, L_B, offsets, idx).reshape(got.shape)
    err = np.abs(got - want)
    assert np.isfinite(got).all() and err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())

    with pytest.raises(ei.EiError):
        pl.debug_waits(wait_limit_log2=99)
