"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

Stages 1-3 are compared with the oracle in full (the oracle's planning stages take well under a
second even at 128k tokens); the attention output is compared on a stratified sample of
(head, segment) cells that the oracle computes one by one on the GPU's own selection.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_09508_b200 as ei
import synth
from synth.generator import with_
from util import bf16_bits_to_f64, lists_of, to_bits, to_dev

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def _sample_cells(wl, rigid, segs):
    hr = np.flatnonzero(rigid)
    hd = np.flatnonzero(~rigid.astype(bool))
    cells = []
    for n, i in enumerate(segs):
        for grp in (hr, hd):
            if len(grp):
                cells.append((int(grp[(7 * n + 3) % len(grp)]), int(i)))
    return cells


def _check_plan(wl, q, k, res, st):
    op = oracle.plan(q, k, wl.L_S, wl.L_B, fraction=wl.fraction)
    e = res["entropy"].astype(np.float64)
    assert (np.abs(e - op.entropy64) <= 1e-3 * np.abs(op.entropy64) + 1e-7).all()
    np.testing.assert_array_equal(res["rigid"], op.rigid)
    np.testing.assert_array_equal(res["rigid"].astype(bool), st.rigid)
    assert res["k"].sum() == op.T
    # budgets: exact given the GPU's own fp32 entropy table; count of cells differing end to end is bounded
    op_tf = oracle.plan(q, k, wl.L_S, wl.L_B, fraction=wl.fraction, entropy_override=res["entropy"])
    np.testing.assert_array_equal(res["k"], op_tf.k)
    n_diff = int((res["k"] != op.k).sum())
    assert n_diff <= max(2, op.k.size // 100), n_diff
    cells = wl.H * wl.C_S
    got = lists_of(res["offsets"], res["idx"], cells)
    want = lists_of(op_tf.offsets, op_tf.idx, cells)
    exempt = 0
    for c in range(cells):
        if not np.array_equal(got[c], want[c]):
            assert op_tf.gap[c] < 1e-4, (c, op_tf.gap[c])
            exempt += 1
    assert exempt <= max(2, cells // 50), exempt
    return n_diff, exempt


def _check_attention(wl, q, k, v, res, out, cells):
    got = bf16_bits_to_f64(to_bits(out)).reshape(wl.H, wl.C_S, wl.L_S, wl.d)
    assert np.isfinite(got).all()
    want = oracle.sparse_attention(q, k, v, wl.L_S, wl.L_B, res["offsets"].astype(np.int64), res["idx"], cells=cells)
    g = np.stack([got[h, i] for h, i in cells])
    err = np.abs(g - want)
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())


def _run(wl, q, k, v, qd=None, kd=None, vd=None):
    qd = to_dev(q) if qd is None else qd
    kd = to_dev(k) if kd is None else kd
    vd = to_dev(v) if vd is None else vd
    out = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
    pl = ei.Plan(ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction))
    pl.plan(qd, kd)
    pl.sparse_prefill(qd, kd, vd, out)
    res = pl.results()
    assert pl.status() == 0
    return res, out, (qd, kd, vd)


def _dynamic_cells(wl, rigid, segs, per_seg=2):
    """Cells of Dynamic heads (diffuse rows: a Rigid cell's output is a copy of V[g, 0] and proves little), two
    heads per listed segment, plus one Rigid cell."""
    hd = np.flatnonzero(~rigid.astype(bool))
    hr = np.flatnonzero(rigid)
    cells = [(int(hd[(5 * n + 3 * m + 1) % len(hd)]), int(i)) for n, i in enumerate(segs) for m in range(per_seg)]
    if len(hr):
        cells.append((int(hr[0]), int(segs[-1])))
    return cells


@pytest.mark.parametrize("name,segs", [
    ("llama3_8b_32k", [1, 9, 40, 63]),
    ("llama3_8b_128k", [2, 30, 90, 127]),
    ("qwen25_7b_64k", [1, 20, 77, 127]),
])
def test_benchmark_workloads_full_size_three_seeds(name, segs):
    # every planning stage in full against the oracle on three seeds (the Qwen shape draws its Rigid fraction from
    # the seed, so the Rigid / Dynamic mix varies); attention on eight Dynamic cells and one Rigid cell of the
    # first seed, on one Dynamic cell of the others
    base = synth.WORKLOADS[name]
    for n, seed in enumerate((base.seed, base.seed + 1, base.seed + 2)):
        wl = with_(base, seed=seed)
        q, k, v, st = synth.generate(wl)
        res, out, _ = _run(wl, q, k, v)
        _check_plan(wl, q, k, res, st)
        cells = _dynamic_cells(wl, res["rigid"], segs) if n == 0 else _dynamic_cells(wl, res["rigid"], segs[1:2], 1)[:1]
        _check_attention(wl, q, k, v, res, out, cells)
        if name == "llama3_8b_128k" and n == 0:
            _check_latent_compress_full_shape(wl, q, k, v)
        del out
        torch.cuda.empty_cache()


def _check_latent_compress_full_shape(wl, q, k, v):
    # Alg. 4 at the benchmarked shape (H 32 / H_kv 8 / d 128 / L 131072, window 64, budget 1024): scores, kept
    # positions and gathered rows of three KV heads against the oracle, with the tolerances of test_gpu_compress
    from test_gpu_compress import check, run_compress
    qw = np.ascontiguousarray(q[:, -64:])
    check(qw, k, v, 1024, run_compress(qw, k, v, 1024), heads=(0, 3, 7))


@pytest.mark.parametrize("rho", [0.2, 0.5, 0.8])
def test_llama31_70b_shape_budget_and_mix_sweep(rho):
    # the 70B-shaped layer at every budget of the sweep {2, 5, 10, 25, 100 %} for one Rigid fraction of {0.2, 0.5,
    # 0.8}: all planning stages in full, attention on sampled cells (early segments where the lists are long)
    base = with_(synth.WORKLOADS["llama31_70b_128k"], rigid_fraction=rho, seed=5000 + int(10 * rho))
    q, k, v, st = synth.generate(base)
    assert int(st.rigid.sum()) == round(rho * base.H)
    dev = None
    prev_k = None
    for f, segs in [(0.02, [3, 127]), (0.05, [40, 100]), (0.10, [17, 64]), (0.25, [3, 8]), (1.0, [0, 4])]:
        wl = with_(base, fraction=f)
        res, out, dev = _run(wl, q, k, v, *(dev or (None, None, None)))
        _check_plan(wl, q, k, res, st)
        if prev_k is not None:
            assert (res["k"] >= prev_k).all()       # budgets grow with the configured total
        prev_k = res["k"]
        if f == 1.0:                                # 100 % = dense: every causal block selected
            Ci = np.array([wl.r * (i + 1) for i in range(wl.C_S)])
            np.testing.assert_array_equal(res["k"], np.broadcast_to(Ci, res["k"].shape))
        _check_attention(wl, q, k, v, res, out, _dynamic_cells(wl, res["rigid"], segs, 1))
        del out
        torch.cuda.empty_cache()


def test_128k_variants_group_shared_ragged_and_chunked():
    # the benchmark sequence once more in the three widened forms, each against the oracle on sampled cells:
    # group-shared lists; a length that is not a multiple of the segment (131072 - 777 tokens); the last 48k
    # positions as a chunk against all keys
    wl = synth.WORKLOADS["llama3_8b_128k"]
    q, k, v, st = synth.generate(wl)
    G = wl.H // wl.Hkv

    def attend(params, qa, ka, va, n_rows):
        pl = ei.Plan(params)
        out = torch.full((wl.H, n_rows, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
        qd, kd, vd = to_dev(qa), to_dev(ka), to_dev(va)
        pl.plan(qd, kd)
        pl.sparse_prefill(qd, kd, vd, out)
        res = pl.results()
        assert pl.status() == 0
        return res, bf16_bits_to_f64(to_bits(out))

    def check_cells(got, qa, ka, va, off, idx, cells, n_rows):
        want = oracle.sparse_attention(qa, ka, va, wl.L_S, wl.L_B, off, idx, cells=cells)
        for n, (h, i) in enumerate(cells):
            rows = slice(i * wl.L_S, min((i + 1) * wl.L_S, n_rows))
            err = np.abs(got[h, rows] - want[n, :rows.stop - rows.start])
            assert np.isfinite(got[h, rows]).all()
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (h, i, err.max(), err.mean())

    # ---- group-shared
    p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
    p.flags = ei.FLAG_GROUP_SHARED
    res, got = attend(p, q, k, v, wl.N)
    want = oracle.plan(q, k, wl.L_S, wl.L_B, fraction=wl.fraction, group_shared=True,
                       entropy_override=res["group_entropy"])
    np.testing.assert_array_equal(res["k"], want.k)
    off_h, idx_h = oracle.expand_group_lists(res["offsets"], res["idx"], wl.Hkv, G, wl.C_S)
    check_cells(got, q, k, v, off_h, idx_h, [(0, 0), (5, 3), (17, 64), (31, 127)], wl.N)

    # ---- ragged length
    N2 = wl.N - 777
    q2, k2, v2 = (np.ascontiguousarray(a[:, :N2]) for a in (q, k, v))
    res, got = attend(ei.params_default(wl.H, wl.Hkv, wl.d, N2, wl.L_S, wl.L_B, wl.fraction), q2, k2, v2, N2)
    want = oracle.plan(q2, k2, wl.L_S, wl.L_B, fraction=wl.fraction, entropy_override=res["entropy"])
    np.testing.assert_array_equal(res["k"], want.k)
    assert int(res["k"].sum()) == want.T
    check_cells(got, q2, k2, v2, res["offsets"].astype(np.int64), res["idx"], [(1, 0), (9, 70), (2, 127), (30, 127)], N2)

    # ---- chunk: the last 48k positions against all keys
    Nq = 48 * 1024
    qc = np.ascontiguousarray(q[:, wl.N - Nq:])
    p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
    p.q_len = Nq
    p.q_stride_head = p.o_stride_head = Nq * wl.d
    res, got = attend(p, qc, k, v, Nq)
    want = oracle.plan(qc, k, wl.L_S, wl.L_B, fraction=wl.fraction, entropy_override=res["entropy"])
    np.testing.assert_array_equal(res["k"], want.k)
    check_cells(got, qc, k, v, res["offsets"].astype(np.int64), res["idx"], [(0, 0), (12, 20), (31, 47)], Nq)


def test_128k_producer_side_pooling():
    # the benchmark shape through ei_rope_pool + ei_plan_pooled: rotated rows against the oracle on sampled
    # (head, segment) cells; representatives against the oracle's pooling of everything the kernel wrote;
    # the plan bit for bit against ei_plan on the rotated tensors
    wl = synth.WORKLOADS["llama3_8b_128k"]
    q, k, v, st = synth.generate(wl)
    cos, sin = synth.rope_tables(wl.N, wl.d)
    qd, kd = to_dev(q), to_dev(k)
    cd, sd = torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda()
    pl = ei.Plan(ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction))
    pl.rope_pool(qd, kd, cd, sd)                                    # in place
    pl.plan_pooled()
    res = pl.results()
    assert pl.status() == 0
    got_q, got_k = to_bits(qd), to_bits(kd)
    for got, src, L, cells in ((got_q, q, wl.L_S, [(0, 0), (13, 37), (31, 127)]), (got_k, k, wl.L_B, [(0, 0), (5, 600), (7, 1023)])):
        for h, i in cells:
            rows = slice(i * L, (i + 1) * L)
            want = oracle.rope(src[h:h + 1, rows], cos[rows], sin[rows])[0]
            a, b = got[h, rows].astype(np.int32), want.astype(np.int32)
            key = lambda x: np.where(x & 0x8000, -(x & 0x7FFF), x)   # noqa: E731
            big = np.abs(bf16_bits_to_f64(want)) > 2.0 ** -10
            assert np.abs(key(a) - key(b))[big].max() <= 1
            assert (a != b).mean() < 1e-3
    qmax, qmin = oracle.pool(got_q, wl.L_S)
    kmax, kmin = oracle.pool(got_k, wl.L_B)
    for item, want in (("QMAX", qmax), ("QMIN", qmin), ("KMAX", kmax), ("KMIN", kmin)):
        np.testing.assert_array_equal(bf16_bits_to_f64(pl.read(item)).reshape(want.shape), want)
    ref = ei.Plan(ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction))
    ref.plan(qd, kd)                                                # the fused schedule, reading Q and K
    rr = ref.results()
    for key_ in ("entropy", "k", "offsets", "idx"):
        np.testing.assert_array_equal(res[key_], rr[key_])


def test_128k_packed_batch_of_unequal_lengths():
    # the benchmark tensors cut into three sequences of 70000 + 40000 + 21072 tokens, packed: the one call must equal
    # per-sequence calls bit for bit, and sampled cells of the ragged middle sequence the oracle's attention
    wl = synth.WORKLOADS["llama3_8b_128k"]
    q, k, v, st = synth.generate(wl)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    lens = [70000, 40000, 21072]
    cu = np.concatenate([[0], np.cumsum(lens)])
    p = ei.params_default(wl.H, wl.Hkv, wl.d, max(lens), wl.L_S, wl.L_B, 0.0)
    p.base_budget_tokens = 2048.0
    p.q_stride_head = p.k_stride_head = p.v_stride_head = p.o_stride_head = wl.N * wl.d
    pl = ei.Plan(p)
    out = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
    pl.prefill_varlen(qd, kd, vd, out, cu)
    assert pl.status() == 0
    got = to_bits(out)
    for b, n in enumerate(lens):
        lo, hi = int(cu[b]), int(cu[b + 1])
        p1 = ei.params_default(wl.H, wl.Hkv, wl.d, n, wl.L_S, wl.L_B, 0.0)
        p1.base_budget_tokens = 2048.0
        p1.q_stride_head = p1.k_stride_head = p1.v_stride_head = p1.o_stride_head = wl.N * wl.d
        ref = ei.Plan(p1)
        o1 = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
        ref.plan(qd[:, lo:hi], kd[:, lo:hi])
        ref.sparse_prefill(qd[:, lo:hi], kd[:, lo:hi], vd[:, lo:hi], o1[:, lo:hi])
        np.testing.assert_array_equal(got[:, lo:hi], to_bits(o1[:, lo:hi].contiguous()))
        if b == 1:
            res = ref.results()
            qs, ks, vs = (np.ascontiguousarray(a[:, lo:hi]) for a in (q, k, v))
            cells = [(0, 0), (11, 17), (31, 39)]                      # segment 39 is the short last one
            want = oracle.sparse_attention(qs, ks, vs, wl.L_S, wl.L_B, res["offsets"].astype(np.int64), res["idx"],
                                           cells=cells)
            g64 = bf16_bits_to_f64(got[:, lo:hi])
            for m, (h, i) in enumerate(cells):
                rows = slice(i * wl.L_S, min((i + 1) * wl.L_S, n))
                err = np.abs(g64[h, rows] - want[m, :rows.stop - rows.start])
                assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (h, i, err.max(), err.mean())
