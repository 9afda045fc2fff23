"""The allocation-free entry point against the plan-based one (collected last on purpose).

ei_entropy_noalloc serves callers that may not allocate device memory -- a host whose own
allocator owns all of HBM, or a loop that cannot take cudaMalloc's device-wide synchronisation --
by keeping its scratch in a fixed device array.  It must give the entropy table that the existing
stage calls (ei_stage_pool + ei_stage_observe on a plan) give, on two calls in a row that reuse
the same scratch with different shapes, and it must refuse shapes the fixed array cannot hold.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_09508_b200 as ei
import synth
from util import to_dev

pytestmark = pytest.mark.gpu

CASES = [
    synth.Workload("na1", 8, 2, 128, 8192, 512, 128, 0.3, 0.5, 2, 3, seed=901),
    synth.Workload("na2", 8, 2, 64, 2048, 128, 64, 0.25, 0.5, 2, 2, seed=902),   # smaller: stale scratch beyond it
]


def _reference_entropy(wl, qd, kd):
    plan = ei.Plan(ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction))
    plan.stage_pool(qd, kd)
    plan.stage_observe()
    return plan.read("ENTROPY").reshape(wl.H, wl.C_S)


def test_noalloc_entropy_matches_plan_path_twice_in_a_row():
    prepared = []
    for wl in CASES:
        q, k, v, st = synth.generate(wl)
        qd, kd = to_dev(q), to_dev(k)
        out = torch.full((wl.H, wl.C_S), float("nan"), dtype=torch.float32, device="cuda")
        prepared.append((wl, qd, kd, out))
    torch.cuda.synchronize()
    # two calls back to back on the same stream, sharing the fixed scratch
    for wl, qd, kd, out in prepared:
        params = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
        ei.entropy_noalloc(params, qd, kd, out)
    torch.cuda.synchronize()
    for wl, qd, kd, out in prepared:
        got = out.cpu().numpy().astype(np.float64)
        want = _reference_entropy(wl, qd, kd).astype(np.float64)
        assert np.isfinite(got).all()
        # the repository's entropy tolerance; the two paths run the same kernels, so in practice equal
        assert (np.abs(got - want) <= 1e-3 * np.abs(want) + 1e-7).all(), np.abs(got - want).max()
    # and once more in the opposite order
    for wl, qd, kd, out in reversed(prepared):
        out.fill_(float("nan"))
        params = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
        ei.entropy_noalloc(params, qd, kd, out)
        torch.cuda.synchronize()
        want = _reference_entropy(wl, qd, kd).astype(np.float64)
        got = out.cpu().numpy().astype(np.float64)
        assert (np.abs(got - want) <= 1e-3 * np.abs(want) + 1e-7).all()


def test_noalloc_entropy_against_the_oracle_and_without_allocating():
    # Not only the same kernels through another door: the table must be the CPU oracle's (fp64, written from the
    # paper) within the entropy tolerance, also for a chunk of queries (q_len < seq_len).  And the property in the
    # entry point's name: the device's free memory is the same after the calls as before them (one call first, so
    # that one-time set-up by the CUDA runtime is not counted).
    wl = CASES[1]
    q, k, v, st = synth.generate(wl)
    qd, kd = to_dev(q), to_dev(k)
    whole = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
    n_q = wl.N // 2                                   # the second half of the sequence as a chunk
    chunk = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
    chunk.q_len = n_q
    chunk.q_stride_head = wl.N * wl.d                 # the chunk's queries sit inside the whole tensor
    out_w = torch.full((wl.H, wl.C_S), float("nan"), dtype=torch.float32, device="cuda")
    out_c = torch.full((wl.H, n_q // wl.L_S), float("nan"), dtype=torch.float32, device="cuda")
    q_chunk = qd[:, wl.N - n_q:, :]
    ei.entropy_noalloc(whole, qd, kd, out_w)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        ei.entropy_noalloc(whole, qd, kd, out_w)
        ei.entropy_noalloc(chunk, q_chunk, kd, out_c)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    want_w = oracle.plan(q, k, wl.L_S, wl.L_B, fraction=wl.fraction).entropy64
    got_w = out_w.cpu().numpy().astype(np.float64)
    assert (np.abs(got_w - want_w) <= 1e-3 * np.abs(want_w) + 1e-7).all(), np.abs(got_w - want_w).max()
    want_c = oracle.plan(q[:, wl.N - n_q:], k, wl.L_S, wl.L_B, fraction=wl.fraction).entropy64
    got_c = out_c.cpu().numpy().astype(np.float64)
    assert want_c.shape == got_c.shape
    assert (np.abs(got_c - want_c) <= 1e-3 * np.abs(want_c) + 1e-7).all(), np.abs(got_c - want_c).max()


def test_noalloc_rejects_shapes_beyond_the_fixed_scratch():
    # 64 heads at 256k tokens needs ~80 MiB of score rows: more than the 32 MiB array
    params = ei.params_default(64, 8, 128, 262144, 1024, 128, 0.05)
    dummy = torch.zeros(16, dtype=torch.float32, device="cuda")
    with pytest.raises(ei.EiError) as e:
        ei.entropy_noalloc(params, dummy, dummy, dummy)
    assert e.value.code == ei.STATUS["SCRATCH_TOO_SMALL"]
    assert "scratch" in str(e.value)
