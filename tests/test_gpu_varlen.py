"""GPU parity for packed batches of unequal lengths (ei_prefill_varlen): every sequence is planned and attended on
its own; the packed call must equal per-sequence calls bit for bit and the oracle within the output tolerances."""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_09508_b200 as ei
import synth
from util import bf16_bits_to_f64, to_bits, to_dev

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3
H, HKV, D, L_S, L_B = 8, 2, 128, 512, 128
LENS = [700, 2304, 0, 389, 1536]                    # ragged, whole segments, empty, shorter than a segment
LENS_TOTAL = [1700, 2304, 0, 3000]                  # TOTAL mode: long enough that half the causal blocks cover the
                                                    # forced diagonal ones


def packed(layout, lens=LENS, seed=150):
    total = sum(lens)
    q, k, v = synth.generate_plain(H, HKV, total, D, seed=seed)     # [heads, total, d]
    if layout == "token_major":                                     # [total, heads, d]
        dev = [to_dev(np.ascontiguousarray(a.transpose(1, 0, 2))) for a in (q, k, v)]
    else:
        dev = [to_dev(a) for a in (q, k, v)]
    return q, k, v, dev


def make_plan(layout, fraction, base_tokens, flags=0, lens=LENS):
    total = sum(lens)
    p = ei.params_default(H, HKV, D, max(lens), L_S, L_B, fraction if base_tokens is None else 0.0)
    if base_tokens is not None:
        p.base_budget_tokens = base_tokens
    p.flags = flags
    if layout == "token_major":
        p.q_stride_tok = p.o_stride_tok = H * D
        p.k_stride_tok = p.v_stride_tok = HKV * D
        p.q_stride_head = p.k_stride_head = p.v_stride_head = p.o_stride_head = D
    else:
        p.q_stride_head = p.k_stride_head = p.v_stride_head = p.o_stride_head = total * D
    return ei.Plan(p)


@pytest.mark.parametrize("layout", ["head_major", "token_major"])
@pytest.mark.parametrize("mode", ["total", "base", "group"])
def test_packed_batch_equals_per_sequence_calls_and_the_oracle(layout, mode):
    lens = LENS if mode == "base" else LENS_TOTAL
    q, k, v, (qd, kd, vd) = packed(layout, lens)
    total = sum(lens)
    fraction, base = (0.5, None) if mode != "base" else (0.0, 640.0)
    flags = ei.FLAG_GROUP_SHARED if mode == "group" else 0
    pl = make_plan(layout, fraction, base, flags, lens)
    out = torch.full(qd.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    cu = np.concatenate([[0], np.cumsum(lens)])
    pl.prefill_varlen(qd, kd, vd, out, cu)
    assert pl.status() == 0
    got = to_bits(out)
    if layout == "token_major":
        got = np.ascontiguousarray(got.reshape(total, H, D).transpose(1, 0, 2))
    got = got.reshape(H, total, D)
    for b, n in enumerate(lens):
        if n == 0:
            continue
        lo, hi = int(cu[b]), int(cu[b + 1])
        qs, ks, vs = (np.ascontiguousarray(a[:, lo:hi]) for a in (q, k, v))
        p1 = ei.params_default(H, HKV, D, n, L_S, L_B, fraction if base is None else 0.0)
        if base is not None:
            p1.base_budget_tokens = base
        p1.flags = flags
        ref = ei.Plan(p1)
        o1 = torch.empty((H, n, D), dtype=torch.bfloat16, device="cuda")
        ref.plan(to_dev(qs), to_dev(ks))
        ref.sparse_prefill(to_dev(qs), to_dev(ks), to_dev(vs), o1)
        np.testing.assert_array_equal(got[:, lo:hi], to_bits(o1).reshape(H, n, D))
        if b in (0, 3):                                                 # oracle parity on the ragged sequences
            res = ref.results()
            C_S = -(-n // L_S)
            off, idx = res["offsets"].astype(np.int64), res["idx"]
            if mode == "group":
                off, idx = oracle.expand_group_lists(off, idx, HKV, H // HKV, C_S)
            want = oracle.sparse_attention(qs, ks, vs, L_S, L_B, off, idx).reshape(H, C_S * L_S, D)[:, :n]
            err = np.abs(bf16_bits_to_f64(got[:, lo:hi]) - want)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())
    last = [n for n in lens if n][-1]
    assert pl.params.seq_len == last and pl.Nq == last           # left targeted at the last sequence


def test_packed_batch_arguments_are_checked():
    q, k, v, (qd, kd, vd) = packed("head_major")
    out = torch.zeros_like(qd)
    pl = make_plan("head_major", 0.0, 640.0)
    with pytest.raises(ei.EiError) as e:
        pl.prefill_varlen(qd, kd, vd, out, [0, 512, 256])           # not monotone
    assert e.value.code == ei.STATUS["INVALID_ARG"]
    with pytest.raises(ei.EiError) as e:
        pl.prefill_varlen(qd, kd, vd, out, [0, 512, 512 + max(LENS) + L_B])   # longer than the plan was made for
    assert e.value.code == ei.STATUS["PLAN_MISMATCH"]
    tot = make_plan("head_major", 0.35, None)
    with pytest.raises(ei.EiError) as e:                             # TOTAL mode: 35 % of a 389-token sequence's
        tot.prefill_varlen(qd, kd, vd, out, [0, 2304, 2304 + 389])    # blocks is fewer than its forced diagonal blocks
    assert e.value.code == ei.STATUS["BUDGET_INFEASIBLE"]
    torch.cuda.synchronize()
    assert not out.any()                                             # nothing was launched
    pl.prefill_varlen(qd, kd, vd, out, [0, 0])                       # an empty batch is fine
    assert pl.status() == 0


@pytest.mark.parametrize("mode", ["total", "base", "group"])
@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_packed_batch_in_one_set_of_launches(mode, layout):
    # A plan made for the batch's total length has room for every sequence's tables side by side: the whole batch
    # then costs five launches (pool, observe, budget, select, attention), however many sequences it has -- and
    # still equals per-sequence calls bit for bit.
    rng = np.random.default_rng(7)
    if mode == "base":
        lens = [int(x) for x in rng.integers(130, 2100, size=11)] + [0, 2048, 129]
    elif mode == "group":
        lens = [int(x) for x in rng.integers(1700, 3000, size=5)] + [0, 2560]
    else:                                               # long enough that half the causal blocks cover the diagonal ones
        lens = [int(x) for x in rng.integers(1700, 3000, size=8)] + [0, 2048, 1701]
    total = sum(lens)
    q, k, v, (qd, kd, vd) = packed(layout, lens, seed=151)
    fraction, base = (0.5, None) if mode != "base" else (0.0, 640.0)
    flags = ei.FLAG_GROUP_SHARED if mode == "group" else 0
    # (room for every sequence's segments: each sequence rounds up to whole segments of its own)
    p = ei.params_default(H, HKV, D, sum(-(-n // L_S) * L_S for n in lens), L_S, L_B, fraction)
    if base is not None:
        p.base_budget_tokens = base
    if layout == "token_major":
        p.q_stride_tok = p.o_stride_tok = H * D
        p.k_stride_tok = p.v_stride_tok = HKV * D
        p.q_stride_head = p.k_stride_head = p.v_stride_head = p.o_stride_head = D
    else:
        p.q_stride_head = p.k_stride_head = p.v_stride_head = p.o_stride_head = total * D
    p.flags = flags
    pl = ei.Plan(p)
    out = torch.full(qd.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    cu = np.concatenate([[0], np.cumsum(lens)])
    n0 = pl.launches()
    pl.prefill_varlen(qd, kd, vd, out, cu)
    assert pl.status() == 0
    assert pl.launches() - n0 == (6 if mode == "group" else 5)     # group-shared lists: one aggregation launch more
    got = to_bits(out)
    if layout == "token_major":
        got = np.ascontiguousarray(got.reshape(total, H, D).transpose(1, 0, 2))
    got = got.reshape(H, total, D)
    for b, n in enumerate(lens):
        if n == 0:
            continue
        lo, hi = int(cu[b]), int(cu[b + 1])
        qs, ks, vs = (np.ascontiguousarray(a[:, lo:hi]) for a in (q, k, v))
        p1 = ei.params_default(H, HKV, D, n, L_S, L_B, fraction)
        if base is not None:
            p1.base_budget_tokens = base
        p1.flags = flags
        ref = ei.Plan(p1)
        o1 = torch.empty((H, n, D), dtype=torch.bfloat16, device="cuda")
        ref.plan(to_dev(qs), to_dev(ks))
        ref.sparse_prefill(to_dev(qs), to_dev(ks), to_dev(vs), o1)
        np.testing.assert_array_equal(got[:, lo:hi], to_bits(o1).reshape(H, n, D), err_msg=f"sequence {b} of {n} tokens")
    with pytest.raises(ei.EiError) as e:                # the tables hold a batch now: nothing to attend from
        pl.sparse_prefill(qd, kd, vd, out)
    assert e.value.code == ei.STATUS["NOT_PLANNED"]


@pytest.mark.parametrize("shape", [(4, 2, 64, 256, 64), (4, 2, 64, 256, 128), (6, 2, 128, 128, 64), (4, 1, 128, 384, 128),
                                   (4, 2, 256, 256, 128), (2, 1, 256, 128, 64)],
                         ids=lambda s_: "H%d_Hkv%d_d%d_LS%d_LB%d" % s_)
def test_packed_batch_in_one_set_of_launches_other_shapes(shape):
    # the same for the shapes that take the two-tile pair kernel (d or L_B = 64, segments a multiple of 256) and the
    # one-tile kernel (other segment lengths, head_dim 256)
    h, hkv, d, ls, lb = shape
    rng = np.random.default_rng(11)
    lens = [int(x) for x in rng.integers(70, 1500, size=7)] + [0, 4 * ls, ls + 1]
    total = sum(lens)
    q, k, v = synth.generate_plain(h, hkv, total, d, seed=152)
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    p = ei.params_default(h, hkv, d, sum(-(-n // ls) * ls for n in lens), ls, lb, 0.0)
    p.base_budget_tokens = 3.0 * lb
    p.q_stride_head = p.k_stride_head = p.v_stride_head = p.o_stride_head = total * d
    pl = ei.Plan(p)
    out = torch.full(qd.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    cu = np.concatenate([[0], np.cumsum(lens)])
    n0 = pl.launches()
    pl.prefill_varlen(qd, kd, vd, out, cu)
    assert pl.status() == 0
    assert pl.launches() - n0 == 5
    got = to_bits(out).reshape(h, total, d)
    for b, n in enumerate(lens):
        if n == 0:
            continue
        lo, hi = int(cu[b]), int(cu[b + 1])
        qs, ks, vs = (np.ascontiguousarray(a[:, lo:hi]) for a in (q, k, v))
        p1 = ei.params_default(h, hkv, d, n, ls, lb, 0.0)
        p1.base_budget_tokens = 3.0 * lb
        ref = ei.Plan(p1)
        o1 = torch.empty((h, n, d), dtype=torch.bfloat16, device="cuda")
        ref.plan(to_dev(qs), to_dev(ks))
        ref.sparse_prefill(to_dev(qs), to_dev(ks), to_dev(vs), o1)
        np.testing.assert_array_equal(got[:, lo:hi], to_bits(o1).reshape(h, n, d), err_msg=f"sequence {b} of {n} tokens")
