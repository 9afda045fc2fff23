"""GPU parity: every stage of the CUDA path against the CPU oracle, through the C ABI.

Stage-isolated checks feed a stage the oracle's output of the previous stage, so that a tolerance
at one stage cannot hide a bug in the next; the end-to-end checks then run the whole path.

Tolerances (the stated tolerances of the method's hot path):
  entropies  |d| <= 1e-3 |e_oracle| + 1e-7
  budgets and block lists bit-exact, except cells whose oracle boundary gap (score of the last
  block taken minus best block left out, in ln A) is below 1e-4
  bf16 output: max-abs 2e-2 and mean-abs 2e-3 against the fp64 oracle on the same selection
"""
import math

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


def make_plan(wl, fraction=None, base_tokens=None, flags=0):
    p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, fraction if fraction else 0.0)
    if base_tokens is not None:
        p.base_budget_tokens = base_tokens
    p.flags = flags
    return ei.Plan(p)


SMALL = {
    "tiny": synth.WORKLOADS["tiny"],
    # d = 128 / L_B = 128 in a size the oracle finishes in seconds; several tiles, ragged lists
    "mid128": synth.Workload("mid128", 8, 2, 128, 4096, 512, 128, 0.30, 0.5, 2, 3, seed=77),
    # GQA 7:1, one KV head
    "gqa7": synth.Workload("gqa7", 7, 1, 128, 2048, 256, 128, 0.40, 0.43, 1, 2, seed=78),
    # d = 128 with 64-wide key blocks, d = 64 with 128-wide key blocks
    "d128b64": synth.Workload("d128b64", 4, 2, 128, 2048, 256, 64, 0.35, 0.5, 2, 2, seed=79),
    "d64b128": synth.Workload("d64b128", 4, 4, 64, 2048, 256, 128, 0.50, 0.5, 1, 1, seed=80),
}


@pytest.fixture(scope="module", params=list(SMALL))
def case(request):
    wl = SMALL[request.param]
    q, k, v, st = synth.generate(wl)
    op = oracle.plan(q, k, wl.L_S, wl.L_B, fraction=wl.fraction)
    return dict(wl=wl, q=q, k=k, v=v, st=st, op=op, qd=to_dev(q), kd=to_dev(k), vd=to_dev(v))


# ------------------------------------------------------------------ stage 1a: pooling (exact)
def test_pool_exact(case):
    wl, op = case["wl"], case["op"]
    pl = make_plan(wl, wl.fraction)
    pl.stage_pool(case["qd"], case["kd"])
    for item, ref in (("QMAX", "qmax"), ("QMIN", "qmin"), ("KMAX", "kmax"), ("KMIN", "kmin")):
        got = bf16_bits_to_f64(pl.read(item)).reshape(op.reps[ref].shape)
        np.testing.assert_array_equal(got, op.reps[ref], err_msg=item)
    assert pl.status() == 0


def test_pool_strided_inputs(case):
    # token stride > d (e.g. q/k/v interleaved in one buffer) must give the same result
    wl, op = case["wl"], case["op"]
    pad = 2 * wl.d
    qbig = torch.zeros((wl.H, wl.N, pad), dtype=torch.bfloat16, device="cuda")
    kbig = torch.zeros((wl.Hkv, wl.N, pad), dtype=torch.bfloat16, device="cuda")
    qbig[..., :wl.d] = case["qd"]
    kbig[..., :wl.d] = case["kd"]
    p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
    p.q_stride_tok = p.k_stride_tok = pad
    p.q_stride_head = p.k_stride_head = wl.N * pad
    pl = ei.Plan(p)
    pl.stage_pool(qbig, kbig)
    got = bf16_bits_to_f64(pl.read("QMAX")).reshape(op.reps["qmax"].shape)
    np.testing.assert_array_equal(got, op.reps["qmax"])
    got = bf16_bits_to_f64(pl.read("KMIN")).reshape(op.reps["kmin"].shape)
    np.testing.assert_array_equal(got, op.reps["kmin"])


# ------------------------------------------------------------------ stage 1b: observation + entropy
def test_observe_entropy_and_scores(case):
    wl, op = case["wl"], case["op"]
    pl = make_plan(wl, wl.fraction)
    pl.stage_pool(case["qd"], case["kd"])
    pl.stage_observe()
    e = pl.read("ENTROPY").reshape(wl.H, wl.C_S).astype(np.float64)
    tol = 1e-3 * np.abs(op.entropy64) + 1e-7
    assert (np.abs(e - op.entropy64) <= tol).all(), np.abs(e - op.entropy64).max()
    # far inside the tolerance on Dynamic heads, so that budgets rarely depend on it
    dyn = ~op.rigid.astype(bool)
    rel = np.abs(e[dyn] - op.entropy64[dyn]) / np.abs(op.entropy64[dyn])
    assert rel.max() < 2e-5, rel.max()
    sc = pl.read("SCORES").reshape(wl.H, -1).astype(np.float64)
    err = np.abs(sc - op.lnA)
    assert err.max() < 5e-5, err.max()
    assert (sc <= 0).all()


# ------------------------------------------------------------------ stage 2: budgets (exact, teacher-forced)
def _budget_roundtrip(wl, e32, fraction=None, base_tokens=None):
    pl = make_plan(wl, fraction, base_tokens)
    pl.write("ENTROPY", e32.ravel())
    pl.stage_budget()
    k = pl.read("BUDGET").reshape(wl.H, wl.C_S)
    rigid = pl.read("CLASS")
    offsets = pl.read("OFFSETS")
    stats = pl.read("STATS")
    assert pl.status() == 0
    return k, rigid, offsets, stats, pl


def test_budget_exact_given_oracle_entropy(case):
    wl, op = case["wl"], case["op"]
    k, rigid, offsets, stats, pl = _budget_roundtrip(wl, op.entropy, fraction=wl.fraction)
    np.testing.assert_array_equal(rigid, op.rigid)
    np.testing.assert_array_equal(k, op.k)
    np.testing.assert_array_equal(offsets, op.offsets)
    assert stats[0] == op.T == pl.total_blocks() and stats[1] == op.rigid.sum() and stats[2] == op.b_star
    assert stats[4] == op.k.min() and stats[5] == op.k.max()


@pytest.mark.parametrize("fraction", [None, 0.02, 0.07, 0.5, 1.0])
def test_budget_exact_on_random_entropy_tables(fraction):
    # tables that reach the 3x cap, zero entries (denominator floor), rigid rows
    wl = synth.Workload("b", 16, 4, 128, 16384, 256, 128, 0.1, 0.5, 1, 1)
    rng = np.random.default_rng(5)
    e = rng.gamma(1.5, 1.0, (wl.H, wl.C_S)).astype(np.float32)
    e[:4] = (rng.random((4, wl.C_S)) * 9e-6).astype(np.float32)   # rigid
    e[4, ::5] = 0.0
    e[5] = np.where(np.arange(wl.C_S) % 2 == 0, 1.0, 2.0)
    rigid_o, m = oracle.multipliers(e)
    if fraction is None:
        want = oracle.budgets_base(m, wl.r, 2048.0 / wl.L_B)
        k, rigid, offsets, stats, _ = _budget_roundtrip(wl, e, base_tokens=2048.0)
    else:
        T = oracle.total_blocks(fraction, wl.H, wl.C_S, wl.r)
        if T < wl.H * wl.C_S * wl.r:
            p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, fraction)
            with pytest.raises(ei.EiError) as err:
                ei.Plan(p)
            assert err.value.code == ei.STATUS["BUDGET_INFEASIBLE"]
            return
        want, b = oracle.budgets_total(m, wl.r, T)
        k, rigid, offsets, stats, _ = _budget_roundtrip(wl, e, fraction=fraction)
        assert stats[2] == b and k.sum() == T
    np.testing.assert_array_equal(rigid, rigid_o)
    np.testing.assert_array_equal(k, want)
    np.testing.assert_array_equal(offsets[1:], np.cumsum(want.ravel()))


# ------------------------------------------------------------------ stage 3: selection (exact, teacher-forced)
def test_select_exact_given_scores(case):
    wl, op = case["wl"], case["op"]
    pl = make_plan(wl, wl.fraction)
    sc32 = op.lnA.astype(np.float32)
    pl.write("SCORES", sc32.ravel())
    pl.write("ENTROPY", op.entropy.ravel())
    pl.stage_budget()
    pl.stage_select()
    res = pl.results()
    np.testing.assert_array_equal(res["k"], op.k)
    # the oracle ranks exactly the fp32 values the kernel saw
    offs, idx, gap = oracle.select(sc32.astype(np.float64), op.k, wl.r)
    np.testing.assert_array_equal(res["idx"], idx)
    assert pl.status() == 0


def test_select_ties_and_extremes():
    wl = synth.Workload("s", 4, 2, 64, 4096, 128, 64, 0.3, 0.5, 1, 1)
    rng = np.random.default_rng(9)
    SC = oracle.row_offset(wl.C_S, wl.r)
    sc = -rng.gamma(2.0, 20.0, (wl.H, SC)).astype(np.float32)
    sc[0, ::3] = -1.0                 # many exact ties
    sc[1] = 0.0                       # everything tied: must take the lowest indices
    sc[2, ::7] = 0.0                  # zeros among negatives
    sc[3] = np.round(sc[3])           # coarse values, many ties, down to -300
    k = np.empty((wl.H, wl.C_S), np.int32)
    for i in range(wl.C_S):
        k[:, i] = rng.integers(wl.r, wl.r * (i + 1) + 1, wl.H)
    k[0, -1] = wl.r                   # nothing but the diagonal
    k[1, -1] = wl.r * wl.C_S          # everything
    offs, idx, gap = oracle.select(sc.astype(np.float64), k, wl.r)
    pl = make_plan(wl, 1.0)
    pl.write("SCORES", sc.ravel())
    pl.write("BUDGET", k.ravel())
    pl.write("OFFSETS", offs.astype(np.int32))
    pl.stage_select()
    got = pl.read("INDICES", count=int(offs[-1]))
    np.testing.assert_array_equal(got, idx)


# ------------------------------------------------------------------ stages 1-3 end to end
def test_plan_end_to_end(case):
    wl, op = case["wl"], case["op"]
    pl = make_plan(wl, wl.fraction)
    pl.plan(case["qd"], case["kd"])
    res = pl.results()
    assert pl.status() == 0
    np.testing.assert_array_equal(res["rigid"], op.rigid)
    np.testing.assert_array_equal(res["rigid"].astype(bool), case["st"].rigid)
    assert res["k"].sum() == op.T
    # budgets: exact whenever the GPU's fp32 entropy table gives the same fixed-point multipliers;
    # check against the oracle run on the GPU's own table (exact), and count e2e differences
    op_tf = oracle.plan(case["q"], case["k"], wl.L_S, wl.L_B, fraction=wl.fraction, entropy_override=res["entropy"])
    np.testing.assert_array_equal(res["k"], op_tf.k)
    n_budget_diff = int((res["k"] != op.k).sum())
    assert n_budget_diff <= max(2, op.k.size // 100), n_budget_diff
    # lists: exact except near-tie cells
    cells = wl.H * wl.C_S
    got = lists_of(res["offsets"], res["idx"], cells)
    want = lists_of(op_tf.offsets, op_tf.idx, cells)
    exempt = 0
    for c in range(cells):
        if np.array_equal(got[c], want[c]):
            continue
        assert op_tf.gap[c] < 1e-4, (c, op_tf.gap[c], got[c], want[c])
        exempt += 1
    assert exempt <= max(2, cells // 50), exempt
    # invariants of the lists themselves
    for c in range(cells):
        i = c % wl.C_S
        lst = got[c]
        assert (np.diff(lst) > 0).all() and lst[-1] < wl.r * (i + 1)
        assert set(range(wl.r * i, wl.r * (i + 1))) <= set(lst.tolist())


# ------------------------------------------------------------------ stage 4: attention
def _attention_check(wl, q, k, v, kcounts, idx, offsets, flags=0, cells=None):
    pl = make_plan(wl, 1.0, flags=flags)
    pl.set_lists(kcounts, idx)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    out = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
    pl.sparse_prefill(qd, kd, vd, out)
    assert pl.status() == 0
    got = bf16_bits_to_f64(to_bits(out)).reshape(wl.H, wl.C_S, wl.L_S, wl.d)
    if cells is None:
        cells = [(h, i) for h in range(wl.H) for i in range(wl.C_S)]
    want = oracle.sparse_attention(q, k, v, wl.L_S, wl.L_B, offsets, idx, cells=cells)
    g = np.stack([got[h, i] for h, i in cells])
    assert np.isfinite(g).all()
    err = np.abs(g - want)
    return err.max(), err.mean()


def _full_lists(wl):
    k = np.array([[wl.r * (i + 1) for i in range(wl.C_S)]] * wl.H, np.int32)
    idx = np.concatenate([np.arange(c, dtype=np.int32) for c in k.ravel()])
    offsets = np.concatenate([[0], np.cumsum(k.ravel())]).astype(np.int64)
    return k, idx, offsets


def _random_lists(wl, rng, p_keep=0.3):
    ks, parts = [], []
    for h in range(wl.H):
        for i in range(wl.C_S):
            cand = np.arange(wl.r * i)
            keep = cand[rng.random(cand.size) < p_keep]
            lst = np.concatenate([keep, np.arange(wl.r * i, wl.r * (i + 1))]).astype(np.int32)
            ks.append(len(lst))
            parts.append(lst)
    k = np.array(ks, np.int32).reshape(wl.H, wl.C_S)
    idx = np.concatenate(parts)
    offsets = np.concatenate([[0], np.cumsum(ks)]).astype(np.int64)
    return k, idx, offsets


ATT_SHAPES = [
    # H, Hkv, d, N, L_S, L_B
    (2, 1, 64, 512, 128, 64),
    (4, 2, 128, 1024, 256, 128),
    (2, 2, 128, 1024, 128, 64),
    (2, 1, 64, 1024, 256, 128),
    (8, 2, 128, 2048, 512, 128),
]


@pytest.mark.parametrize("shape", ATT_SHAPES)
@pytest.mark.parametrize("flags", [0, ei.FLAG_ATTN_P_VIA_SMEM, ei.FLAG_ATTN_SINGLE_TILE, ei.FLAG_ATTN_PAIR_8WARP,
                                   ei.FLAG_ATTN_PERSISTENT, ei.FLAG_ATTN_PER_CTA, ei.FLAG_ATTN_SPLIT,
                                   ei.FLAG_ATTN_SPLIT | ei.FLAG_ATTN_NO_SKIP,
                                   ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_NO_SKIP, ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_PERSISTENT,
                                   ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_PERSISTENT | ei.FLAG_ATTN_NO_SKIP,
                                   ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_SINGLE_TILE,
                                   ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_SINGLE_TILE | ei.FLAG_ATTN_NO_SKIP,
                                   ei.FLAG_ATTN_TRI, ei.FLAG_ATTN_TRI | ei.FLAG_ATTN_NO_SKIP])
@pytest.mark.parametrize("lists", ["full", "random", "diag"])
def test_attention_on_plain_inputs(shape, flags, lists):
    # structure-free N(0,1) inputs: diffuse softmax rows in every head, every diagonal-mask case
    H, Hkv, d, N, L_S, L_B = shape
    wl = synth.Workload("a", H, Hkv, d, N, L_S, L_B, 1.0, 0.0, 0, 0)
    q, k, v = synth.generate_plain(H, Hkv, N, d, seed=21 + d + N)
    rng = np.random.default_rng(3)
    if lists == "full":
        kc, idx, offsets = _full_lists(wl)
    elif lists == "random":
        kc, idx, offsets = _random_lists(wl, rng)
    else:
        kc, idx, offsets = _random_lists(wl, rng, p_keep=0.0)
    mx, mean = _attention_check(wl, q, k, v, kc, idx, offsets, flags)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)


@pytest.mark.parametrize("flags", [0, ei.FLAG_ATTN_SINGLE_TILE, ei.FLAG_ATTN_PAIR_8WARP, ei.FLAG_ATTN_PERSISTENT,
                                   ei.FLAG_ATTN_PER_CTA, ei.FLAG_ATTN_SPLIT,
                                   ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_PERSISTENT, ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_SINGLE_TILE,
                                   ei.FLAG_ATTN_TRI])
@pytest.mark.parametrize("which", ["second_diag_only", "empty"])
def test_attention_rows_without_visible_keys(flags, which):
    # hand-made lists in which some (or all) 128-row tiles see no key at all: those rows must come
    # out as zeros, the others as usual (covers the empty-tile paths of every kernel)
    H, Hkv, d, N, L_S, L_B = 2, 1, 128, 1024, 256, 128
    wl = synth.Workload("a", H, Hkv, d, N, L_S, L_B, 1.0, 0.0, 0, 0)
    q, k, v = synth.generate_plain(H, Hkv, N, d, seed=31)
    if which == "empty":
        kc = np.zeros((H, wl.C_S), np.int32)
        idx = np.zeros(0, np.int32)
    else:
        kc = np.ones((H, wl.C_S), np.int32)
        idx = np.array([wl.r * i + 1 for _ in range(H) for i in range(wl.C_S)], np.int32)
    offsets = np.concatenate([[0], np.cumsum(kc.ravel())]).astype(np.int64)
    mx, mean = _attention_check(wl, q, k, v, kc, idx, offsets, flags)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)


def test_attention_full_budget_equals_dense_definition():
    H, Hkv, d, N, L_S, L_B = 4, 2, 128, 1024, 256, 128
    wl = synth.Workload("a", H, Hkv, d, N, L_S, L_B, 1.0, 0.0, 0, 0)
    q, k, v = synth.generate_plain(H, Hkv, N, d, seed=5)
    kc, idx, offsets = _full_lists(wl)
    pl = make_plan(wl, 1.0)
    pl.set_lists(kc, idx)
    out = torch.empty((H, N, d), dtype=torch.bfloat16, device="cuda")
    pl.sparse_prefill(to_dev(q), to_dev(k), to_dev(v), out)
    got = bf16_bits_to_f64(to_bits(out))
    want = oracle.dense_attention(q, k, v)
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())


def test_attention_large_logits_do_not_overflow():
    # logits of several hundred (as in sink heads) stress the online softmax's running max
    H, Hkv, d, N, L_S, L_B = 2, 1, 128, 1024, 256, 128
    wl = synth.Workload("a", H, Hkv, d, N, L_S, L_B, 1.0, 0.0, 0, 0)
    q, k, v = synth.generate_plain(H, Hkv, N, d, seed=6, scale=6.0)
    v = synth.generate_plain(H, Hkv, N, d, seed=7)[2]
    kc, idx, offsets = _full_lists(wl)
    mx, mean = _attention_check(wl, q, k, v, kc, idx, offsets)
    assert mx <= MAX_ABS and mean <= MEAN_ABS, (mx, mean)


def test_whole_path_on_planted_workload(case):
    # ei_plan + ei_sparse_prefill; output compared with the oracle on the GPU's own selection
    wl = case["wl"]
    pl = make_plan(wl, wl.fraction)
    out = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
    pl.plan(case["qd"], case["kd"])
    pl.sparse_prefill(case["qd"], case["kd"], case["vd"], out)
    res = pl.results()
    assert pl.status() == 0
    got = bf16_bits_to_f64(to_bits(out)).reshape(wl.H, wl.C_S, wl.L_S, wl.d)
    want = oracle.sparse_attention(case["q"], case["k"], case["v"], wl.L_S, wl.L_B,
                                   res["offsets"].astype(np.int64), res["idx"])
    want = want.reshape(wl.H, wl.C_S, wl.L_S, wl.d)
    err = np.abs(got - want)
    assert np.isfinite(got).all()
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())
    # run-twice determinism
    out2 = torch.empty_like(out)
    pl.sparse_prefill(case["qd"], case["kd"], case["vd"], out2)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))


def test_prefill_host_matches_device_path(case):
    wl = case["wl"]
    pl = make_plan(wl, wl.fraction)
    out_dev = torch.empty((wl.H, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
    pl.plan(case["qd"], case["kd"])
    pl.sparse_prefill(case["qd"], case["kd"], case["vd"], out_dev)
    out_host = np.empty((wl.H, wl.N, wl.d), np.uint16)
    pl2 = make_plan(wl, wl.fraction)
    pl2.prefill_host(case["q"], case["k"], case["v"], out_host)
    np.testing.assert_array_equal(out_host, to_bits(out_dev))


@pytest.mark.parametrize("flags", [0, ei.FLAG_GROUP_SHARED], ids=["per_head", "group_shared"])
def test_prefill_host_in_base_mode_pipelines_kv_groups(flags):
    # BASE mode: the host path runs every KV group through a plan of its own; same bits as the device path,
    # also when called again (the per-group plans are reused) and on a ragged length
    wl = SMALL["mid128"]
    q, k, v, st = synth.generate(wl)
    for n in (wl.N, wl.N - 300):
        qs, ks, vs = (np.ascontiguousarray(a[:, :n]) for a in (q, k, v))
        p = ei.params_default(wl.H, wl.Hkv, wl.d, n, wl.L_S, wl.L_B, 0.0)
        p.base_budget_tokens = 3.0 * wl.L_B
        p.flags = flags
        dev = ei.Plan(p)
        out_dev = torch.empty((wl.H, n, wl.d), dtype=torch.bfloat16, device="cuda")
        dev.plan(to_dev(qs), to_dev(ks))
        dev.sparse_prefill(to_dev(qs), to_dev(ks), to_dev(vs), out_dev)
        host = ei.Plan(p)
        for rep in range(2):
            out_host = np.zeros((wl.H, n, wl.d), np.uint16)
            host.prefill_host(qs, ks, vs, out_host)
            assert host.status() == 0
            np.testing.assert_array_equal(out_host, to_bits(out_dev))


@pytest.mark.parametrize("persistent", [False, True], ids=["per_cta", "persistent"])
def test_negligible_half_rows_shortcut(persistent):
    # the split-row kernels write P = 0 without exponentials where a warp's half rows lie 24 binary orders below the
    # row maximum.  On diffuse rows only masked half rows qualify (exactly zero either way): bit-identical to the
    # kernel with every probability evaluated.  On the planted workload (Rigid heads with a sink that outweighs
    # everything) most half rows qualify: both forms stay inside the output tolerance and within 1e-4 of each other.
    base = ei.FLAG_ATTN_PERSISTENT if persistent else ei.FLAG_ATTN_PER_CTA
    wl = SMALL["mid128"]
    for planted in (False, True):
        if planted:
            q, k, v, st = synth.generate(wl)
        else:
            q, k, v = synth.generate_plain(wl.H, wl.Hkv, wl.N, wl.d, seed=91)
        qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
        outs = []
        for flags in (base, base | ei.FLAG_ATTN_NO_SKIP):
            pl = make_plan(wl, wl.fraction, flags=flags)
            pl.plan(qd, kd)
            out = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
            pl.sparse_prefill(qd, kd, vd, out)
            assert pl.status() == 0
            outs.append(to_bits(out))
            res = pl.results()
        if not planted:
            np.testing.assert_array_equal(outs[0], outs[1])
            continue
        a, b = bf16_bits_to_f64(outs[0]), bf16_bits_to_f64(outs[1])
        assert np.abs(a - b).max() <= 1e-4
        want = oracle.sparse_attention(q, k, v, wl.L_S, wl.L_B, res["offsets"].astype(np.int64), res["idx"]).reshape(a.shape)
        for got in (a, b):
            err = np.abs(got - want)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())


def test_zero_p_products_left_out_is_bit_identical():
    # EI_FLAG_ATTN_SKIP_ZERO_PV: a P.V product whose P is all zero adds nothing, so leaving it out changes no bit;
    # the counter says how many were left out (many on the planted workload, whose Rigid heads see a sink; none on
    # diffuse rows apart from nothing at all: a masked half does not make a whole tile zero)
    wl = SMALL["mid128"]
    for planted in (True, False):
        if planted:
            q, k, v, st = synth.generate(wl)
        else:
            q, k, v = synth.generate_plain(wl.H, wl.Hkv, wl.N, wl.d, seed=92)
        qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
        outs, left = [], []
        for flags in (ei.FLAG_ATTN_SPLIT, ei.FLAG_ATTN_SKIP_ZERO_PV, ei.FLAG_ATTN_SKIP_ZERO_PV | ei.FLAG_ATTN_NO_SKIP):
            pl = make_plan(wl, wl.fraction, flags=flags)
            pl.plan(qd, kd)
            out = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
            pl.sparse_prefill(qd, kd, vd, out)
            assert pl.status() == 0
            outs.append(to_bits(out))
            left.append(int(pl.read("STATS")[6]))
        np.testing.assert_array_equal(outs[0], outs[1])
        assert left[0] == 0 and left[2] == 0            # not asked for / nothing is ever zeroed without the shortcut
        assert (left[1] > 0) == planted, left


def test_sparse_prefill_requires_a_plan():
    wl = SMALL["tiny"]
    pl = make_plan(wl, wl.fraction)
    t = torch.zeros((wl.H, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
    tk = torch.zeros((wl.Hkv, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ei.EiError) as e:
        pl.sparse_prefill(t, tk, tk, t)
    assert e.value.code == ei.STATUS["NOT_PLANNED"]
    with pytest.raises(ei.EiError) as e:
        pl.set_lists(np.full((wl.H, wl.C_S), 1, np.int32), np.zeros(3, np.int32))
    assert e.value.code == ei.STATUS["PLAN_MISMATCH"]


# ------------------------------------------------------------------ edge cases of the whole path
EDGE = {
    # one segment only (C_S = 1): nothing but diagonal blocks, every budget forced
    "one_segment": (synth.Workload("e1", 4, 2, 128, 512, 512, 128, 1.0, 0.5, 1, 1, seed=91), dict(fraction=1.0)),
    # L_S = L_B (r = 1) and multi-head attention without grouping (G = 1)
    "r1_mha": (synth.Workload("e2", 4, 4, 128, 2048, 128, 128, 0.4, 0.5, 1, 2, seed=92), dict(fraction=0.4)),
    # the smallest feasible total: exactly the forced diagonal blocks
    "min_total": (synth.Workload("e3", 4, 2, 64, 2048, 256, 64, 0.0, 0.5, 1, 1, seed=93), dict(fraction="min")),
    # the paper's own mode: base budget in tokens, no configured total
    "base_2048": (synth.Workload("e4", 8, 2, 128, 8192, 512, 128, 0.0, 0.5, 2, 3, seed=94), dict(base_tokens=2048.0)),
    "base_small": (synth.Workload("e5", 8, 2, 128, 4096, 256, 128, 0.0, 0.5, 2, 3, seed=95), dict(base_tokens=300.0)),
}


@pytest.mark.parametrize("name", list(EDGE))
def test_whole_path_edge_cases(name):
    wl, mode = EDGE[name]
    q, k, v, st = synth.generate(wl)
    kw = {}
    if "base_tokens" in mode:
        kw["base_tokens"] = mode["base_tokens"]
        p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, 0.0)
        p.base_budget_tokens = mode["base_tokens"]
    else:
        f = mode["fraction"]
        if f == "min":   # the fraction whose rounded total is exactly H * C_S * r
            f = (wl.H * wl.C_S * wl.r) / (wl.H * wl.sum_causal)
        kw["fraction"] = f
        p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, f)
    pl = ei.Plan(p)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    out = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
    pl.plan(qd, kd)
    pl.sparse_prefill(qd, kd, vd, out)
    res = pl.results()
    assert pl.status() == 0
    op = oracle.plan(q, k, wl.L_S, wl.L_B, entropy_override=res["entropy"], **kw)
    np.testing.assert_array_equal(res["rigid"], op.rigid)
    np.testing.assert_array_equal(res["k"], op.k)
    cells = wl.H * wl.C_S
    got, want = lists_of(res["offsets"], res["idx"], cells), lists_of(op.offsets, op.idx, cells)
    for c in range(cells):
        assert np.array_equal(got[c], want[c]) or op.gap[c] < 1e-4, c
    if name == "min_total":
        assert (res["k"] == wl.r).all()
    if "base_tokens" in mode:   # k <= 3 B_h / L_B (Alg. 3's cap) and the work bound of Eq. t_spa
        assert (res["k"] <= max(wl.r, 3 * mode["base_tokens"] / wl.L_B)).all()
        assert (res["k"].astype(np.int64).sum(axis=1) * wl.L_B * wl.L_S <= 3 * max(mode["base_tokens"], wl.L_S) * wl.N).all()
    want_o = oracle.sparse_attention(q, k, v, wl.L_S, wl.L_B, res["offsets"].astype(np.int64), res["idx"])
    got_o = bf16_bits_to_f64(to_bits(out)).reshape(want_o.shape)
    err = np.abs(got_o - want_o)
    assert np.isfinite(got_o).all() and err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())


@pytest.mark.parametrize("flags", [0, ei.FLAG_ATTN_SINGLE_TILE, ei.FLAG_ATTN_PAIR_8WARP, ei.FLAG_ATTN_PERSISTENT,
                                   ei.FLAG_ATTN_PER_CTA, ei.FLAG_ATTN_SPLIT,
                                   ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_PERSISTENT, ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_SINGLE_TILE,
                                   ei.FLAG_ATTN_TRI])
def test_attention_strided_tensors(flags):
    # q, k, v and out as views into wider buffers (token stride 3*d, as in a fused QKV activation)
    H, Hkv, d, N, L_S, L_B = 4, 2, 128, 1024, 256, 128
    wl = synth.Workload("a", H, Hkv, d, N, L_S, L_B, 1.0, 0.0, 0, 0)
    q, k, v = synth.generate_plain(H, Hkv, N, d, seed=41)
    rng = np.random.default_rng(4)
    kc, idx, offsets = _random_lists(wl, rng)
    pad = 3 * d
    bufq = torch.zeros((H, N, pad), dtype=torch.bfloat16, device="cuda")
    bufkv = torch.zeros((Hkv, N, pad), dtype=torch.bfloat16, device="cuda")
    bufo = torch.full((H, N, pad), float("nan"), dtype=torch.bfloat16, device="cuda")
    bufq[..., :d] = to_dev(q)
    bufkv[..., d:2 * d] = to_dev(k)
    bufkv[..., 2 * d:] = to_dev(v)
    p = ei.params_default(H, Hkv, d, N, L_S, L_B, 1.0)
    p.flags = flags
    p.q_stride_tok = p.k_stride_tok = p.v_stride_tok = p.o_stride_tok = pad
    p.q_stride_head = p.k_stride_head = p.v_stride_head = p.o_stride_head = N * pad
    pl = ei.Plan(p)
    pl.set_lists(kc, idx)
    pl.sparse_prefill(bufq, bufkv[..., d:], bufkv[..., 2 * d:], bufo[..., d:])
    assert pl.status() == 0
    got = bf16_bits_to_f64(to_bits(bufo[..., d:2 * d].contiguous())).reshape(H, wl.C_S, L_S, d)
    want = oracle.sparse_attention(q, k, v, L_S, L_B, offsets, idx).reshape(H, wl.C_S, L_S, d)
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())
    # nothing outside the output view was written
    assert torch.isnan(bufo[..., :d].float()).all() and torch.isnan(bufo[..., 2 * d:].float()).all()



def test_batch_of_equal_length_sequences_as_stacked_heads():
    # A batch of B equal-length sequences is the same problem with B*H query heads and B*H_kv KV heads
    # (q [B, H, N, d] viewed as [B*H, N, d]: query head b*H + h reads KV head b*H_kv + h / G).  In BASE mode
    # every head is planned on its own, so the stacked call must give exactly the per-sequence results.
    wl = SMALL["d128b64"]
    B = 2
    seqs = [synth.generate(with_(wl, seed=wl.seed + b)) for b in range(B)]
    q = np.concatenate([s[0] for s in seqs])
    k = np.concatenate([s[1] for s in seqs])
    v = np.concatenate([s[2] for s in seqs])
    big = with_(wl, H=B * wl.H, Hkv=B * wl.Hkv)
    pl = make_plan(big, base_tokens=512.0)
    out = torch.empty((big.H, big.N, big.d), dtype=torch.bfloat16, device="cuda")
    pl.plan(to_dev(q), to_dev(k))
    pl.sparse_prefill(to_dev(q), to_dev(k), to_dev(v), out)
    res = pl.results()
    assert pl.status() == 0
    for b in range(B):
        one = make_plan(wl, base_tokens=512.0)
        o1 = torch.empty((wl.H, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
        qb, kb, vb = (to_dev(a) for a in seqs[b][:3])
        one.plan(qb, kb)
        one.sparse_prefill(qb, kb, vb, o1)
        r1 = one.results()
        np.testing.assert_array_equal(res["k"][b * wl.H:(b + 1) * wl.H], r1["k"])
        np.testing.assert_array_equal(res["entropy"][b * wl.H:(b + 1) * wl.H], r1["entropy"])
        np.testing.assert_array_equal(to_bits(out[b * wl.H:(b + 1) * wl.H]), to_bits(o1))


def test_unsupported_head_dim_padded_with_zero_columns():
    # head_dim 96 is refused; padded to 128 with zero columns and with both logit scales set to 1/sqrt(96)
    # it is the d = 96 problem exactly: pooled zeros add nothing to a logit, and the added output columns are 0.
    H, Hkv, N, d, dp, L_S, L_B = 4, 2, 2048, 96, 128, 256, 128
    with pytest.raises(Exception):
        ei.Plan(ei.params_default(H, Hkv, d, N, L_S, L_B, 0.4))
    q, k, v = synth.generate_plain(H, Hkv, N, d, seed=96)
    pad = lambda a: np.concatenate([a, np.zeros(a.shape[:2] + (dp - d,), np.uint16)], axis=2)
    op = oracle.plan(q, k, L_S, L_B, fraction=0.4)
    p = ei.params_default(H, Hkv, dp, N, L_S, L_B, 0.4)
    p.obs_scale = p.attn_scale = 1.0 / math.sqrt(d)
    pl = ei.Plan(p)
    qd, kd, vd = to_dev(pad(q)), to_dev(pad(k)), to_dev(pad(v))
    out = torch.full((H, N, dp), float("nan"), dtype=torch.bfloat16, device="cuda")
    pl.plan(qd, kd)
    pl.sparse_prefill(qd, kd, vd, out)
    res = pl.results()
    assert pl.status() == 0
    e = op.entropy64
    assert (np.abs(res["entropy"] - e) <= 1e-3 * np.abs(e) + 1e-7).all()
    op_tf = oracle.plan(q, k, L_S, L_B, fraction=0.4, entropy_override=res["entropy"])
    np.testing.assert_array_equal(res["k"], op_tf.k)
    cells = H * (N // L_S)
    got, want = lists_of(res["offsets"], res["idx"], cells), lists_of(op_tf.offsets, op_tf.idx, cells)
    for c in range(cells):
        assert np.array_equal(got[c], want[c]) or op_tf.gap[c] < 1e-4, c
    o = bf16_bits_to_f64(to_bits(out))
    assert (o[:, :, d:] == 0).all()
    ref = oracle.sparse_attention(q, k, v, L_S, L_B, res["offsets"], res["idx"]).reshape(H, N, d)
    err = np.abs(o[:, :, :d] - ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())


def test_plan_and_attention_replay_from_a_cuda_graph():
    # ei_plan + ei_sparse_prefill make no synchronising call and allocate nothing after ei_plan_create, so a step
    # can be captured once and replayed; the replay must give the eager result bit for bit, also on new inputs
    # written into the same buffers
    wl = SMALL["mid128"]
    q, k, v, st = synth.generate(wl)
    q2, k2, v2, _ = synth.generate(with_(wl, seed=wl.seed + 1))
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    pl = make_plan(wl, wl.fraction)
    out = torch.zeros((wl.H, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        pl.plan(qd, kd, stream=side)                      # warm-up outside the capture (function attributes are set)
        pl.sparse_prefill(qd, kd, vd, out, stream=side)
    side.synchronize()
    eager = to_bits(out).copy()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        pl.plan(qd, kd, stream=side)
        pl.sparse_prefill(qd, kd, vd, out, stream=side)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_bits(out), eager)
    qd.copy_(to_dev(q2)); kd.copy_(to_dev(k2)); vd.copy_(to_dev(v2))
    graph.replay()
    torch.cuda.synchronize()
    replayed = to_bits(out).copy()
    pl2 = make_plan(wl, wl.fraction)
    out2 = torch.empty_like(out)
    pl2.plan(qd, kd)
    pl2.sparse_prefill(qd, kd, vd, out2)
    np.testing.assert_array_equal(replayed, to_bits(out2))
    assert pl.status() == 0


@pytest.mark.parametrize("name", ["tiny", "mid128", "gqa7", "d64b128"])
def test_fused_and_staged_planning_agree_bit_for_bit(name):
    # the persistent pool + observe kernel must leave exactly what the stage kernels leave: pooled representatives,
    # scores, entropies, and therefore budgets and lists (small shapes pick the staged schedule on their own, so the
    # fused one is forced here; the full-size tests run it by default)
    wl = SMALL[name]
    q, k, v, st = synth.generate(wl)
    qd, kd = to_dev(q), to_dev(k)
    got = []
    for flags in (ei.FLAG_PLAN_STAGED, ei.FLAG_PLAN_FUSED):
        pl = make_plan(wl, wl.fraction, flags=flags)
        pl.plan(qd, kd)
        assert pl.status() == 0
        got.append({it: pl.read(it) for it in ("QMAX", "QMIN", "KMAX", "KMIN", "ENTROPY", "SCORES", "BUDGET", "OFFSETS")}
                   | {"idx": pl.results()["idx"]})
    for key in got[0]:
        np.testing.assert_array_equal(got[0][key], got[1][key], err_msg=key)


@pytest.mark.parametrize("name", ["mid128", "gqa7"])
def test_forms_of_a_kernel_family_agree_bit_for_bit(name):
    # same arithmetic per tile, only the assignment of tiles to CTAs differs: the quad-layout kernels (one CTA per
    # tile pair = the library's own choice, persistent, one tile per CTA) agree among themselves, and so do the two
    # split-row kernels; two launches in a row also check that the item counter is back at zero after a launch
    wl = SMALL[name]
    q, k, v, st = synth.generate(wl)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    families = [(0, ei.FLAG_ATTN_PER_CTA, ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_PERSISTENT, ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_SINGLE_TILE),
                (ei.FLAG_ATTN_SPLIT, ei.FLAG_ATTN_PERSISTENT)]
    for family in families:
        for group in (0, ei.FLAG_GROUP_SHARED):
            outs = []
            for flags in family:
                pl = make_plan(wl, wl.fraction, flags=flags | group)
                pl.plan(qd, kd)
                for rep in range(2):
                    out = torch.full((wl.H, wl.N, wl.d), float("nan"), dtype=torch.bfloat16, device="cuda")
                    pl.sparse_prefill(qd, kd, vd, out)
                    assert pl.status() == 0
                    outs.append(to_bits(out))
            for o in outs[1:]:
                np.testing.assert_array_equal(outs[0], o)
