"""Pins for the CPU oracle: it is checked against what the paper and the mathematics fix, never against itself.

Each test names the passage it pins.  None of them needs a GPU.
"""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from paper_2609_00097_b200.workloads import make_workload, repage

HERE = os.path.dirname(os.path.abspath(__file__))
CODEBOOK = np.array([-1.5, -0.5, 0.5, 1.5])   # App. A.1, printed
INF = float("inf")


def bf16_bits(x):
    """float array -> bf16 bit patterns (values must already be bf16-representable or are rounded by torch)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# ---------------------------------------------------------------------------------------------------------
# number formats: pinned to numpy's IEEE conversions
# ---------------------------------------------------------------------------------------------------------

def test_fp16_decode_matches_numpy_exhaustively(oracle):
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([oracle.fp16_value(int(b)) for b in bits])
    both_nan = np.isnan(want) & np.isnan(got)
    assert np.all((want == got) | both_nan)
    assert math.copysign(1.0, oracle.fp16_value(0x8000)) == -1.0


def test_fp16_rounding_matches_numpy(oracle):
    rng = np.random.default_rng(5)
    xs = np.concatenate([
        np.abs(rng.standard_normal(20000)).astype(np.float32) * np.float32(3.0),
        (10.0 ** rng.uniform(-9, 4.8, 20000)).astype(np.float32),
        np.arange(0, 2048, dtype=np.float32) * np.float32(2.0 ** -25),          # subnormal ties
        np.array([0.0, 65504.0, 65503.9, 2.0 ** -24, 2.0 ** -25, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11],
                 dtype=np.float32),
    ])
    xs = xs[xs <= 65504.0]
    want = xs.astype(np.float16).view(np.uint16)
    got = np.array([oracle.fp16_round(float(x)) for x in xs], dtype=np.uint16)
    assert np.array_equal(want, got)


def test_bf16_decode_matches_numpy(oracle):
    bits = np.arange(0, 65536, 7, dtype=np.uint16)
    want = bits_to_f64(bits)
    got = np.array([oracle.bf16_value(int(b)) for b in bits])
    ok = (want == got) | (np.isnan(want) & np.isnan(got))
    assert np.all(ok)


# ---------------------------------------------------------------------------------------------------------
# App. A.1: quantizer
# ---------------------------------------------------------------------------------------------------------

def _one_column(values_bits):
    """A cache of one page, one head, BLK = len(values), D = 1 holding the given bf16 column."""
    n = len(values_bits)
    return values_bits.reshape(1, 1, n, 1).copy(), np.array([n], dtype=np.int32)


@pytest.mark.parametrize("absmax", [1.5, 2.71875, 0.01226806640625, 1000.0, 3.0e-5])
def test_codes_equal_argmin_over_all_bf16_values(oracle, absmax):
    """App. A.1: x_q = argmin_c |x/s - c| with s = max|x|/1.5, checked on every bf16 value below the maximum."""
    allbits = np.arange(65536, dtype=np.uint16)
    vals = bits_to_f64(allbits)
    keep = np.isfinite(vals) & (np.abs(vals) <= absmax)
    column = np.concatenate([allbits[keep], bf16_bits([absmax])])
    k, seq = _one_column(column)
    codes, scales = oracle.quantize(k, None, seq, 1)
    x = bits_to_f64(column)
    # printed scale rule, evaluated by numpy in the stated precisions
    want_scale = (np.float32(absmax) / np.float32(1.5)).astype(np.float16)
    assert scales[0, 0, 0] == want_scale.view(np.uint16)
    s = float(want_scale)
    dist = np.abs(x[:, None] / s - CODEBOOK[None, :])
    order = np.sort(dist, axis=1)
    clear = (order[:, 1] - order[:, 0]) > 1e-9
    got = codes[0, 0, :, 0]
    assert np.array_equal(got[clear], np.argmin(dist, axis=1)[clear])
    # where fp64 cannot separate the two nearest levels (tiny |x|, or x next to a decision point) evaluate the
    # arg-min in exact rational arithmetic; only exact ties are left out
    fs = Fraction(s)
    levels = [Fraction(-3, 2), Fraction(-1, 2), Fraction(1, 2), Fraction(3, 2)]
    exact_ties = 0
    for i in np.where(~clear)[0]:
        d = [abs(Fraction(float(x[i])) / fs - c) for c in levels]
        best = min(d)
        winners = [j for j in range(4) if d[j] == best]
        if len(winners) > 1:
            exact_ties += 1
            continue
        assert got[i] == winners[0], (x[i], got[i], winners)
    assert exact_ties <= 6                                       # x in {+-0, +-s} (and nothing else)
    # the stated tie rule: |x| = s goes to the outer level, +-0 to +0.5
    ties = {s: 3, -s: 0, 0.0: 2}
    for v, c in ties.items():
        idx = np.where(x == v)[0]                               # +-s is present only when s is a bf16 value
        assert len(idx) > 0 or v != 0.0
        assert np.all(got[idx] == c), (v, got[idx])
    negzero = np.where(column == 0x8000)[0]
    assert np.all(got[negzero] == 2)


def test_quantizer_roundtrip_bound_and_extremes(oracle):
    """Mid-rise grid: every reconstruction is a non-zero level times s; |x - x_hat| <= s/2 up to the fp16
    rounding of s (bound s*(0.5 + 1.5*2^-10)); the absmax element maps to +-1.5 s."""
    w = make_workload("C1", N=1024, tail=13)
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    K = bits_to_f64(w.bits("k_cache"))
    S = scales.view(np.float16).astype(np.float64)[:, :, None, :]
    nb = w.num_blocks(0)
    for blk in range(nb):
        rows = min(64, int(w.seq_lens[0]) - 64 * blk)
        k = K[blk, :, :rows]
        c = codes[blk, :, :rows]
        s = S[blk]
        a = np.abs(k).max(axis=1, keepdims=True)
        assert np.array_equal(scales[blk].view(np.float16),
                              (a[:, 0].astype(np.float32) / np.float32(1.5)).astype(np.float16))
        khat = (c.astype(np.float64) - 1.5) * s
        assert np.all(np.abs(khat) >= 0.5 * s - 1e-12)          # zero-free grid
        assert np.all(np.abs(k - khat) <= s * (0.5 + 1.5 * 2.0 ** -10) + 1e-12)
        at_max = np.abs(k) == a
        assert np.all(np.abs(khat[at_max]) == np.broadcast_to(1.5 * s, k.shape)[at_max])
        assert np.all(np.sign(khat[k != 0]) == np.sign(k[k != 0]))


def test_padding_rows_do_not_move_the_scale(oracle):
    w = make_workload("C1", N=512, tail=40)
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    k2 = w.bits("k_cache").copy()
    last = w.num_blocks(0) - 1
    rows = int(w.seq_lens[0]) - 64 * last
    assert np.all(bits_to_f64(k2[last, :, rows:]) > 9000)       # the generator's poison is there
    k2[last, :, rows:] = bf16_bits([-3.0e4])[0]
    codes2, scales2 = oracle.quantize(k2, w.block_table, w.seq_lens, w.max_blocks)
    assert np.array_equal(scales, scales2)
    assert np.array_equal(codes[:, :, :rows], codes2[:, :, :rows])
    assert scales.view(np.float16).astype(np.float64).max() < 10.0


# ---------------------------------------------------------------------------------------------------------
# hand-worked example (tests/golden/worked_example.json)
# ---------------------------------------------------------------------------------------------------------

# ---------------------------------------------------------------------------------------------------------
# Sec. 3.1 / Alg. 1 Dequant / Sec. 3.3 two-term score: the 8-bit residual
# ---------------------------------------------------------------------------------------------------------

def _full_key(codes, scales, k_res):
    """Alg. 1 Dequant, by numpy: level * s + residual * s / 254."""
    S = scales.view(np.float16).astype(np.float64)[:, :, None, :]
    return (codes.astype(np.float64) - 1.5) * S + k_res.astype(np.float64) * S / 254.0


def test_residual_brings_the_key_back_to_half_a_step(oracle):
    """Sec. 3.1: kept keys are rebuilt to near-16-bit precision.  With an 8-bit symmetric grid over the 2-bit cell
    [-s/2, s/2] every valid element comes back to within half a step, s/508 (+ the binary32 roundings, 1e-6 s):
    about 1/760 of the block's largest key, 250 times closer than the 2-bit level alone.  A wrong sign, channel or
    token index in the residual breaks the bound at once."""
    w = make_workload("C1", N=1024, tail=13)
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    k_res = oracle.quantize_residual(w.bits("k_cache"), codes, scales, w.block_table, w.seq_lens, w.max_blocks)
    assert k_res.dtype == np.int8 and k_res.min() >= -127
    K = bits_to_f64(w.bits("k_cache"))
    full = _full_key(codes, scales, k_res)
    S = np.broadcast_to(scales.view(np.float16).astype(np.float64)[:, :, None, :], K.shape)
    n = int(w.seq_lens[0])
    for blk in range(w.num_blocks(0)):
        rows = min(64, n - 64 * blk)
        err = np.abs(full[blk, :, :rows] - K[blk, :, :rows])
        assert np.all(err <= S[blk, :, :rows] * (1.0 / 508.0 + 1e-6))
        assert np.all(k_res[blk, :, rows:] == 0)                          # padding rows
        # the grid is used: codes reach the ends of the range and are not all tiny
        if rows == 64:
            assert np.abs(k_res[blk]).max() >= 120
    # and the residual really is the finer part: the 2-bit level alone is ~ s/4 off on average
    lvl_err = np.abs((codes.astype(np.float64) - 1.5) * S - K)[: w.num_blocks(0) - 1]
    res_err = np.abs(full - K)[: w.num_blocks(0) - 1]
    assert res_err.mean() < lvl_err.mean() / 100


def test_two_term_score_equals_the_exact_score_when_the_residual_is_exact(oracle):
    """Sec. 3.3: s_final = (q.k_quant + q.k_res) / sqrt(d) is the Dequant form of Alg. 1, and it equals q.k / sqrt(d)
    when the residual loses nothing.  Construction: every channel's largest key is +-0.75, so s = 0.5 and the levels
    are +-0.25, +-0.75; every key is a level plus -127, 0 or +127 residual steps of s / 254, i.e. a multiple of 0.25
    (a bf16 value).  The test checks these premises itself, then asks for identical results from both refinements."""
    rng = np.random.default_rng(12)
    P, Hkv, G = 6, 2, 2
    s = 0.5
    level = rng.choice(CODEBOOK, size=(P, Hkv, 64, 128)) * s
    steps = rng.choice(np.array([-127, 0, 127]), size=(P, Hkv, 64, 128))
    K = np.clip(level + steps * s / 254.0, -0.75, 0.75)
    rows = rng.integers(0, 64, size=(P, Hkv, 128))
    pp, hh, cc = np.meshgrid(np.arange(P), np.arange(Hkv), np.arange(128), indexing="ij")
    K[pp, hh, rows, cc] = 0.75 * rng.choice([-1.0, 1.0], size=(P, Hkv, 128))
    kb = bf16_bits(K)
    assert np.array_equal(bits_to_f64(kb), K)                  # premise: every key is a bf16 value
    seq = np.array([64 * P], dtype=np.int32)
    codes, scales = oracle.quantize(kb, None, seq, P)
    assert np.all(scales.view(np.float16) == np.float16(0.5))  # premise: s = 0.5 in every channel
    k_res = oracle.quantize_residual(kb, codes, scales, None, seq, P)
    assert set(np.unique(k_res).tolist()) == {-127, 0, 127}
    assert np.array_equal(_full_key(codes, scales, k_res), K)  # premise: the residual is exact
    q = bf16_bits(rng.standard_normal((1, Hkv * G, 128)) * 4.0)
    v = bf16_bits(rng.standard_normal((P, Hkv, 64, 128)))
    for delta in (0.5, 6.0, INF):
        a = oracle.decode(q, kb, v, codes, scales, None, seq, P, delta, n_sink=1, n_local=1)
        b = oracle.decode(q, kb, v, codes, scales, None, seq, P, delta, n_sink=1, n_local=1, k_res=k_res)
        assert np.array_equal(a.kept, b.kept)
        assert np.abs(a.out - b.out).max() < 1e-12 and np.abs(a.lse - b.lse).max() < 1e-12
    # and a residual that is wrong by one step in one element is seen
    k_bad = k_res.copy()
    k_bad[0, 0, 0, 0] += 1 if k_bad[0, 0, 0, 0] < 127 else -1
    c = oracle.decode(q, kb, v, codes, scales, None, seq, P, INF, n_sink=1, n_local=1, k_res=k_bad)
    assert np.abs(c.lse[0, :G] - a.lse[0, :G]).max() > 0


def test_residual_refinement_stays_within_its_logit_bound_of_the_exact_one(oracle):
    """With an inexact residual every refined logit moves by at most sm * sum_c |q_c| s_c / 508 (half a step per
    channel); softmax weights then move by at most a factor exp(2 * that), so the output stays close."""
    w = make_workload("C1", N=2048, tail=7)
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    k_res = oracle.quantize_residual(w.bits("k_cache"), codes, scales, w.block_table, w.seq_lens, w.max_blocks)
    a = oracle.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table, w.seq_lens,
                      w.max_blocks, 6.0)
    b = oracle.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table, w.seq_lens,
                      w.max_blocks, 6.0, k_res=k_res)
    assert np.array_equal(a.kept, b.kept) and np.array_equal(a.block_max, b.block_max)   # selection is untouched
    q = np.abs(bits_to_f64(w.bits("q")))[0]                                              # [Hq, D]
    S = scales.view(np.float16).astype(np.float64)                                       # [pages, Hkv, D]
    G = w.Hq // w.Hkv
    bound = max(float((q[h] * S[:, h // G].max(axis=0)).sum()) for h in range(w.Hq)) / 508.0 / math.sqrt(128)
    assert bound < 0.1                                     # worst case; errors of random sign stay far below it
    vmax = np.abs(bits_to_f64(w.bits("v_cache"))).max()
    assert np.abs(a.lse - b.lse).max() <= bound + 1e-12
    assert np.abs(a.lse - b.lse).max() <= bound / 10
    assert np.abs(a.out - b.out).max() <= (math.exp(2 * bound) - 1) * vmax
    assert np.abs(a.out - b.out).max() > 0                                               # and it is not the same path


def test_residual_worked_column_zero_channel_and_saturation(oracle):
    """One column by hand.  Largest key a = 3.015625: s = fp16(a / 1.5) = 2.009765625 (rounded down), step s / 254.
    a -> level 1.5 s = 3.0146484, 0.12 steps short: 0.  2.0 < s -> level 0.5 s = 1.0048828, 125.77 steps: 126.
    0 -> level +0.5 s, exactly -127 steps.  0.125 -> -111.2 steps: -111.  An all-zero channel has s = 0: residual 0.
    A key beyond the saturated scale (|x| > 1.5 * 65504) pins the residual at +-127 instead of wrapping."""
    col = bf16_bits(np.array([3.015625, -3.015625, 2.0, -2.0, 0.0] + [0.125] * 59))
    k, seq = _one_column(col)
    codes, scales = oracle.quantize(k, None, seq, 1)
    assert float(scales.view(np.float16)[0, 0, 0]) == 2.009765625
    res = oracle.quantize_residual(k, codes, scales, None, seq, 1)[0, 0, :, 0]
    assert res[:5].tolist() == [0, 0, 126, -126, -127] and np.all(res[5:] == -111)
    k, seq = _one_column(bf16_bits(np.zeros(64)))
    codes, scales = oracle.quantize(k, None, seq, 1)
    assert np.all(oracle.quantize_residual(k, codes, scales, None, seq, 1) == 0)
    k, seq = _one_column(bf16_bits(np.array([1.0e6, -1.0e6, 98304.0, 1.0] + [0.0] * 60)))
    codes, scales = oracle.quantize(k, None, seq, 1)
    assert float(scales.view(np.float16)[0, 0, 0]) == 65504.0
    res = oracle.quantize_residual(k, codes, scales, None, seq, 1)[0, 0, :, 0]
    assert res[0] == 127 and res[1] == -127 and res[2] == 0     # 98304 - 98256 = 48 = 0.19 steps of 65504 / 254


@pytest.fixture(scope="module")
def golden():
    with open(os.path.join(HERE, "golden", "worked_example.json")) as f:
        return json.load(f)


def _run_golden(oracle, g, case, delta, V=None):
    K = np.array(case["K"], dtype=np.float32)                    # [nb, BLK, D]
    nb, BLK, D = K.shape
    k = bf16_bits(K).reshape(nb, 1, BLK, D)
    v = bf16_bits(np.full((nb, 1, BLK, D), 100.0) if V is None else V).reshape(nb, 1, BLK, D)
    q = bf16_bits(np.array(case["q"], dtype=np.float32)).reshape(1, 1, D)
    seq = np.array([nb * BLK], dtype=np.int32)
    codes, scales = oracle.quantize(k, None, seq, nb)
    r = oracle.decode(q, k, v, codes, scales, None, seq, nb, delta, n_sink=g["n_sink"], n_local=g["n_local"],
                      sm_scale=g["sm_scale"])
    return codes, scales, r


def test_golden_case_a_codes_scores_masks(oracle, golden):
    case = golden["case_A"]
    codes, scales, r = _run_golden(oracle, golden, case, 3.0)
    assert np.array_equal(codes[:, 0], np.array(case["codes"], dtype=np.uint8))
    assert np.all(scales == case["scale_fp16_bits"])
    assert np.array_equal(r.block_max[0, 0], np.array(case["block_max"]))
    assert r.mtilde[0, 0] == case["mtilde"]
    for d, want in case["kept"].items():
        _, _, rr = _run_golden(oracle, golden, case, float(d))
        assert list(rr.kept[0, 0]) == want, d


def test_golden_case_a_output_is_softmax_over_kept_tokens(oracle, golden):
    case = golden["case_A"]
    nb, BLK, D = np.array(case["K"]).shape
    V = np.full((nb, BLK, D), 100.0, dtype=np.float32)
    for j, (blk, row) in enumerate(case["V_onehot_tokens"]):
        V[blk, row] = 0.0
        V[blk, row, j] = 1.0
    _, _, r = _run_golden(oracle, golden, case, case["delta_for_output"], V=V)
    w = np.exp(np.array(case["exponents"]))
    assert np.allclose(r.out[0, 0], w / w.sum(), rtol=0, atol=1e-15)
    assert abs(r.lse[0, 0] - (case["lse_offset"] + math.log(w.sum()))) < 1e-14


def test_golden_case_b_delta_is_a_natural_log_gap_on_scaled_scores(oracle, golden):
    """Eq. 1-2 and the printed constants: a token exactly delta = 5 below the peak carries e^-5 of the peak's
    weight, printed as about 0.67 % and about 1/148."""
    case = golden["case_B"]
    for d, want in case["kept"].items():
        _, _, rr = _run_golden(oracle, golden, case, float(d))
        assert list(rr.kept[0, 0]) == want, d
        assert np.array_equal(rr.block_max[0, 0], np.array(case["block_max"]))
    nb, BLK, D = np.array(case["K"]).shape
    V = np.zeros((nb, BLK, D), dtype=np.float32)
    V[tuple(case["peak_token"])][0] = 1.0
    V[tuple(case["threshold_token"])][1] = 1.0
    _, _, r = _run_golden(oracle, golden, case, 5.0, V=V)
    ratio = r.out[0, 0, 1] / r.out[0, 0, 0]
    assert abs(ratio * 100 - case["printed_ratio_percent"]) < 0.005
    assert round(1.0 / ratio) == case["printed_ratio_inverse"]
    assert abs(1.0 / math.exp(-7.0) - 1096) < 1.0                # the second printed constant


# ---------------------------------------------------------------------------------------------------------
# dense attention and delta = +inf against a library routine
# ---------------------------------------------------------------------------------------------------------

def _torch_dense(w):
    """softmax(q K^T / sqrt(d)) V by torch's scaled_dot_product_attention in fp64 (GQA by repetition)."""
    outs = []
    for b in range(w.B):
        N = int(w.seq_lens[b])
        pages = [w.page(b, blk) for blk in range(w.num_blocks(b))]
        K = w.k_cache[pages].double().permute(1, 0, 2, 3).reshape(w.Hkv, -1, 128)[:, :N]
        V = w.v_cache[pages].double().permute(1, 0, 2, 3).reshape(w.Hkv, -1, 128)[:, :N]
        K = K.repeat_interleave(w.G, dim=0)
        V = V.repeat_interleave(w.G, dim=0)
        q = w.q[b].double().unsqueeze(1)
        outs.append(torch.nn.functional.scaled_dot_product_attention(q, K, V).squeeze(1))
    return torch.stack(outs).numpy()


@pytest.mark.parametrize("name,kw", [("C1", dict(N=1500)), ("C5", dict(B=3, lens=(300, 900)))])
def test_dense_and_delta_inf_equal_library_softmax_attention(oracle, name, kw):
    w = make_workload(name, **kw)
    want = _torch_dense(w)
    out, lse = oracle.dense(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), w.block_table, w.seq_lens,
                            w.max_blocks)
    assert np.abs(out - want).max() < 1e-12
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    r = oracle.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table, w.seq_lens,
                      w.max_blocks, INF)
    assert np.abs(r.out - want).max() < 1e-12
    assert np.abs(r.lse - lse).max() < 1e-12
    for b in range(w.B):
        assert np.all(r.kept[b, :, : w.num_blocks(b)] == 1)
        assert np.all(r.kept[b, :, w.num_blocks(b):] == 0)


# ---------------------------------------------------------------------------------------------------------
# Alg. 1 re-derived by brute force on small inputs (numpy matrices, written from the algorithm box)
# ---------------------------------------------------------------------------------------------------------

def _brute_force(w, codes, scales, delta, n_sink, n_local, bits=2):
    levels = np.arange(1 << bits) - ((1 << bits) - 1) / 2.0       # {-1.5 .. 1.5}, {-7.5 .. 7.5}, {-127.5 .. 127.5}
    B, Hq, G = w.B, w.Hq, w.G
    out = np.zeros((B, Hq, 128))
    kept = np.zeros((B, Hq, w.max_blocks), dtype=np.uint8)
    mt = np.zeros((B, Hq))
    Kc = bits_to_f64(w.bits("k_cache"))
    Vc = bits_to_f64(w.bits("v_cache"))
    Q = bits_to_f64(w.bits("q"))
    S = scales.view(np.float16).astype(np.float64)
    for b in range(B):
        N = int(w.seq_lens[b])
        nb = w.num_blocks(b)
        pages = [w.page(b, i) for i in range(nb)]
        for h in range(Hq):
            g = h // G
            Khat = np.concatenate([levels[codes[p, g]] * S[p, g][None, :] for p in pages])[:N]
            approx = Khat @ Q[b, h] / math.sqrt(128)
            token_block = np.arange(N) // 64
            bm = np.array([approx[token_block == i].max() for i in range(nb)])
            S_set = [i for i in range(nb) if i < n_sink or i >= nb - n_local]
            m = max(bm[i] for i in S_set)
            sel = bm >= m - delta
            kept[b, h, :nb] = sel
            mt[b, h] = m
            Kx = np.concatenate([Kc[p, g] for p in pages])[:N]
            Vx = np.concatenate([Vc[p, g] for p in pages])[:N]
            tok = sel[token_block]
            logits = Kx[tok] @ Q[b, h] / math.sqrt(128)
            p_ = np.exp(logits - logits.max())
            out[b, h] = (p_ / p_.sum()) @ Vx[tok]
    return out, kept, mt


@pytest.mark.parametrize("delta", [0.0, 2.0, 6.0])
def test_decode_equals_brute_force_on_small_inputs(oracle, delta):
    w = make_workload("C5", B=3, lens=(700, 2600), variant=2)      # ragged tails, paged, GQA 4
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    r = oracle.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table, w.seq_lens,
                      w.max_blocks, delta, n_sink=1, n_local=4)
    out, kept, mt = _brute_force(w, codes, scales, delta, 1, 4)
    assert np.abs(r.mtilde - mt).max() < 1e-11
    assert np.array_equal(r.kept, kept)
    assert np.abs(r.out - out).max() < 1e-11


# ---------------------------------------------------------------------------------------------------------
# the deeper thumbnails of the quantization-depth appendix (4 and 8 bits): same construction, 2^b levels
# ---------------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("absmax", [7.5, 2.71875, 1000.0, 3.0e-4])
def test_deeper_codes_equal_argmin_over_all_bf16_values(oracle, bits, absmax):
    """The mid-rise construction of App. A.1 with 2^b levels +-(k + 1/2) and s = max|x| / (2^(b-1) - 1/2): every bf16
    value below the maximum takes the nearest level (arg-min, in exact rational arithmetic where double cannot tell),
    ties go outward; the scale is the stated quotient in the stated precisions."""
    absmax = float(bits_to_f64(bf16_bits([absmax]))[0])          # (the nearest bf16 value)
    allbits = np.arange(65536, dtype=np.uint16)
    vals = bits_to_f64(allbits)
    keep = np.isfinite(vals) & (np.abs(vals) <= absmax)
    column = np.concatenate([allbits[keep][::3], bf16_bits([absmax, -absmax, 0.0])])
    k, seq = _one_column(column)
    codes, scales = oracle.quantize(k, None, seq, 1, bits=bits)
    top = (1 << (bits - 1)) - 0.5
    want_scale = (np.float32(absmax) / np.float32(top)).astype(np.float16)
    assert scales[0, 0, 0] == want_scale.view(np.uint16)
    s = float(want_scale)
    levels = np.arange(1 << bits) - ((1 << bits) - 1) / 2.0
    x = bits_to_f64(column)
    got = codes[0, 0, :, 0].astype(np.int64)
    assert got.min() >= 0 and got.max() <= (1 << bits) - 1
    dist = np.abs(x[:, None] / s - levels[None, :])
    order = np.sort(dist, axis=1)
    clear = (order[:, 1] - order[:, 0]) > 1e-9
    assert np.array_equal(got[clear], np.argmin(dist, axis=1)[clear])
    fs = Fraction(s)
    flevels = [Fraction(int(2 * l), 2) for l in levels]
    ties = 0
    for i in np.where(~clear)[0]:
        d = [abs(Fraction(float(x[i])) / fs - c) for c in flevels]
        best = min(d)
        winners = [j for j in range(len(flevels)) if d[j] == best]
        if len(winners) > 1:      # an exact tie |x| = k s: outward (the level of larger magnitude); +-0: +1/2
            ties += 1
            want = max(winners, key=lambda j: (abs(flevels[j]), flevels[j]))
            assert got[i] == want, (x[i], got[i], winners)
            continue
        assert got[i] == winners[0], (x[i], got[i], winners)
    assert ties >= 2                                              # +0 and -0 at least
    assert got[-3] == (1 << bits) - 1 and got[-2] == 0            # the absmax element takes the outermost level, either sign


@pytest.mark.parametrize("bits", [4, 8])
def test_deeper_roundtrip_bound_and_worked_column(oracle, bits):
    """Half a step: |x - level * s| <= s/2 up to the fp16 rounding of s, on a workload; and a column worked by hand."""
    w = make_workload("C1", N=1024, tail=13)
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks, bits=bits)
    K = bits_to_f64(w.bits("k_cache"))
    S = scales.view(np.float16).astype(np.float64)[:, :, None, :]
    off = ((1 << bits) - 1) / 2.0
    top = (1 << (bits - 1)) - 0.5
    for blk in range(w.num_blocks(0)):
        rows = min(64, int(w.seq_lens[0]) - 64 * blk)
        k, c, s = K[blk, :, :rows], codes[blk, :, :rows].astype(np.float64), S[blk]
        assert np.all(np.abs(k - (c - off) * s) <= s * (0.5 + top * 2.0 ** -10))
        a = np.abs(k).max(axis=1, keepdims=True)
        assert np.array_equal(scales[blk].view(np.float16), (a[:, 0].astype(np.float32) / np.float32(top)).astype(np.float16))
    # by hand, 4 bits: absmax 15 -> s = 2; cells [0,2) -> +0.5, [2,4) -> +1.5, ..., [14, inf) -> +7.5
    col = bf16_bits([15.0, 0.0, 1.99, 2.0, -2.0, -1.0, 13.9, 14.0, -15.0, 7.0, -7.0])
    k, seq = _one_column(col)
    c4, s4 = oracle.quantize(k, None, seq, 1, bits=4)
    assert s4.view(np.float16)[0, 0, 0] == np.float16(2.0)
    assert c4[0, 0, :, 0].tolist() == [15, 8, 8, 9, 6, 7, 14, 15, 0, 11, 4]
    # 8 bits: absmax 255 -> s = 2; x = 3 lies in [2, 4): level +1.5 = code 129
    col = bf16_bits([255.0, 3.0, -3.0, 0.5, -255.0])
    k, seq = _one_column(col)
    c8, s8 = oracle.quantize(k, None, seq, 1, bits=8)
    assert s8.view(np.float16)[0, 0, 0] == np.float16(2.0)
    assert c8[0, 0, :, 0].tolist() == [255, 129, 126, 128, 0]


@pytest.mark.parametrize("bits", [4, 8])
def test_deeper_decode_equals_brute_force_and_tightens_the_scan(oracle, bits):
    """Alg. 1 with deeper thumbnails against the numpy matrix form; and what the appendix's premise needs: more bits
    bring the approximate block maxima closer to the exact ones."""
    w = make_workload("C5", B=3, lens=(700, 2600), variant=2)
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks, bits=bits)
    r = oracle.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table, w.seq_lens,
                      w.max_blocks, 6.0, n_sink=1, n_local=4, bits=bits)
    out, kept, mt = _brute_force(w, codes, scales, 6.0, 1, 4, bits=bits)
    assert np.abs(r.mtilde - mt).max() < 1e-10
    assert np.array_equal(r.kept, kept)
    assert np.abs(r.out - out).max() < 1e-10
    # exact block maxima (16-bit keys) against the approximate ones of 2 bits and of `bits` bits
    Kc, Q = bits_to_f64(w.bits("k_cache")), bits_to_f64(w.bits("q"))
    c2, s2 = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    r2 = oracle.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), c2, s2, w.block_table, w.seq_lens,
                       w.max_blocks, 6.0, n_sink=1, n_local=4)
    err2 = errb = 0.0
    for b in range(w.B):
        for blk in range(w.num_blocks(b)):
            rows = min(64, int(w.seq_lens[b]) - 64 * blk)
            for h in range(0, w.Hq, 5):
                exact = (Kc[w.page(b, blk), h // w.G, :rows] @ Q[b, h]).max() / math.sqrt(128)
                err2 += abs(r2.block_max[b, h, blk] - exact)
                errb += abs(r.block_max[b, h, blk] - exact)
    assert errb < err2 / 3


# ---------------------------------------------------------------------------------------------------------
# properties of the selection rule and of the output
# ---------------------------------------------------------------------------------------------------------

@pytest.fixture(scope="module")
def small(oracle):
    w = make_workload("C2", N=6000)
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    return w, codes, scales


def _decode(oracle, w, codes, scales, delta, **kw):
    return oracle.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, w.block_table,
                         w.seq_lens, w.max_blocks, delta, **kw)


def test_planted_needles_are_kept_and_most_blocks_are_skipped(oracle, small):
    w, codes, scales = small
    r = _decode(oracle, w, codes, scales, 6.0)
    nb = w.num_blocks(0)
    for (b, g), blocks in w.needles.items():
        assert len(blocks) >= 2
        for h in range(g * w.G, (g + 1) * w.G):
            for blk in blocks:
                assert r.kept[b, h, blk] == 1
    assert r.kept[:, :, :nb].mean() < 0.1


def test_mask_monotone_in_delta_nonempty_and_superset_of_global_max_rule(oracle, small):
    """Sec. 5.2: the pseudo-max never exceeds the global approximate max, so the kept set contains the one
    the global-max rule would keep; the block that attains the pseudo-max always passes (delta >= 0)."""
    w, codes, scales = small
    nb = w.num_blocks(0)
    prev = None
    for delta in [0.0, 1.0, 4.0, 6.0, 8.0, 30.0, INF]:
        r = _decode(oracle, w, codes, scales, delta)
        k = r.kept[0, :, :nb].astype(bool)
        assert np.all(k.sum(-1) >= 1)
        gmax = r.block_max[0, :, :nb].max(-1)
        assert np.all(r.mtilde[0] <= gmax + 1e-15)
        if np.isfinite(delta):
            would = r.block_max[0, :, :nb] >= (gmax[:, None] - delta)
            assert np.all(k | ~would)
        if prev is not None:
            assert np.all(k | ~prev)
        prev = k
    assert np.all(prev)
    # no-sink variant: the pseudo-max underestimates and the rule falls back to keeping (almost) everything
    w2 = make_workload("C2", N=6000, sink=False)
    c2, s2 = oracle.quantize(w2.bits("k_cache"), None, w2.seq_lens, w2.max_blocks)
    r2 = _decode(oracle, w2, c2, s2, 6.0)
    assert r2.kept[0, :, :nb].mean() > 0.9


def test_selection_rule_variants_against_their_definitions(oracle):
    """The comparison rules next to Alg. 1's pseudo-max (Fig. 1, Sec. 4.4 "Selection-Rule Overhead", Sec. 5.2).  The block
    maxima are pinned elsewhere; here each rule's kept set is re-derived from them with numpy (sorting, accumulate) and the
    rules are ordered as the mathematics says: global max  subset of  running max  subset of  pseudo-max."""
    cases = [make_workload("C4", N=16384),                      # no sink needle: m_tilde below the global maximum
             make_workload("C5", B=3, lens=(700, 3000)),        # paged, ragged
             make_workload("C2", N=6000)]                       # sink needle: the three threshold rules coincide
    strict = 0
    for w in cases:
        codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
        for delta in (0.0, 3.0, 6.0):
            base = _decode(oracle, w, codes, scales, delta)
            glob = _decode(oracle, w, codes, scales, delta, rule=oracle.RULE_GLOBAL_MAX)
            run = _decode(oracle, w, codes, scales, delta, rule=oracle.RULE_RUNNING_MAX)
            assert np.array_equal(base.block_max, glob.block_max) and np.array_equal(base.block_max, run.block_max)
            for b in range(w.B):
                nb = w.num_blocks(b)
                bm = base.block_max[b, :, :nb]
                mt = base.mtilde[b][:, None]
                assert np.array_equal(glob.kept[b, :, :nb], (bm >= bm.max(-1, keepdims=True) - delta).astype(np.uint8))
                ref = np.maximum(np.maximum.accumulate(bm, axis=-1), mt)
                assert np.array_equal(run.kept[b, :, :nb], (bm >= ref - delta).astype(np.uint8))
                assert np.array_equal(run.thr[b, :, :nb], ref - delta)
                g, r_, p_ = (x.kept[b, :, :nb].astype(bool) for x in (glob, run, base))
                assert np.all(r_ | ~g) and np.all(p_ | ~r_)
                strict += int((p_ & ~r_).sum() > 0) + int((r_ & ~g).sum() > 0)
                # the block attaining the global maximum survives every rule
                arg = bm.argmax(-1)
                for x in (glob, run, base):
                    assert np.all(x.kept[b, np.arange(w.Hq), arg] == 1)
            # the outputs are the exact attention over each rule's own mask
            forced = _decode(oracle, w, codes, scales, delta, forced_mask=run.kept)
            assert np.array_equal(forced.out, run.out) and np.array_equal(forced.lse, run.lse)
        # fixed budget: exactly k blocks when the k-th and (k+1)-th maxima differ, the k largest ones; k >= nb keeps all
        for k in (1, 5, 40):
            top = _decode(oracle, w, codes, scales, 6.0, rule=oracle.RULE_TOP_K, top_k=k)
            for b in range(w.B):
                nb = w.num_blocks(b)
                bm = top.block_max[b, :, :nb]
                order = np.sort(bm, axis=-1)[:, ::-1]
                tau = order[:, min(k, nb) - 1] if k < nb else np.full(w.Hq, -np.inf)
                want = bm >= tau[:, None]
                assert np.array_equal(top.kept[b, :, :nb], want.astype(np.uint8))
                distinct = (k >= nb) | (order[:, min(k, nb - 1)] < tau)
                assert np.all(want.sum(-1)[distinct] == min(k, nb)) and np.all(want.sum(-1) >= min(k, nb))
        everything = _decode(oracle, w, codes, scales, 0.0, rule=oracle.RULE_TOP_K, top_k=10 ** 6)
        dense_o, dense_l = oracle.dense(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), w.block_table, w.seq_lens,
                                        w.max_blocks)
        assert np.abs(everything.out - dense_o).max() < 1e-12
    assert strict >= 4, "the cases never separated the three threshold rules"
    w = cases[2]
    codes, scales = oracle.quantize(w.bits("k_cache"), w.block_table, w.seq_lens, w.max_blocks)
    with pytest.raises(ValueError):
        _decode(oracle, w, codes, scales, 6.0, rule=oracle.RULE_TOP_K, top_k=0)
    with pytest.raises(ValueError):
        _decode(oracle, w, codes, scales, 6.0, rule=7)


def test_delta_zero_keeps_the_pseudo_max_block(oracle, small):
    w, codes, scales = small
    nb = w.num_blocks(0)
    r = _decode(oracle, w, codes, scales, 0.0)
    in_S = np.array([i < 1 or i >= nb - 16 for i in range(nb)])
    for h in range(w.Hq):
        bm = r.block_max[0, h, :nb]
        arg = int(np.argmax(np.where(in_S, bm, -np.inf)))
        assert r.kept[0, h, arg] == 1
        assert bm[arg] == r.mtilde[0, h]


def test_constant_values_give_constant_output_and_output_stays_in_range(oracle, small):
    w, codes, scales = small
    v2 = w.bits("v_cache").copy()
    v2[...] = bf16_bits([0.75])[0]
    r = oracle.decode(w.bits("q"), w.bits("k_cache"), v2, codes, scales, None, w.seq_lens, w.max_blocks, 6.0)
    assert np.abs(r.out - 0.75).max() < 1e-12
    r = _decode(oracle, w, codes, scales, 6.0)
    V = bits_to_f64(w.bits("v_cache"))
    nb = w.num_blocks(0)
    for h in range(0, w.Hq, 5):
        g = h // w.G
        blocks = np.where(r.kept[0, h, :nb])[0]
        rows = np.concatenate([V[blk, g, : min(64, 6000 - 64 * blk)] for blk in blocks])
        assert np.all(r.out[0, h] <= rows.max(0) + 1e-12) and np.all(r.out[0, h] >= rows.min(0) - 1e-12)


def test_sparse_lse_below_dense_lse_and_close_output(oracle, small):
    w, codes, scales = small
    r = _decode(oracle, w, codes, scales, 6.0)
    out, lse = oracle.dense(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), None, w.seq_lens, w.max_blocks)
    assert np.all(r.lse <= lse + 1e-12)
    cos = (r.out * out).sum(-1) / np.linalg.norm(r.out, axis=-1) / np.linalg.norm(out, axis=-1)
    assert cos.min() > 0.999                                      # Sec. 5.1 recall metric on needle data


def test_single_kept_block_closed_form(oracle, small):
    w, codes, scales = small
    forced = np.zeros((1, w.Hq, w.max_blocks), dtype=np.uint8)
    blk = 17
    forced[:, :, blk] = 1
    r = _decode(oracle, w, codes, scales, 6.0, forced_mask=forced)
    K = w.k_cache[blk].double()
    V = w.v_cache[blk].double()
    for h in range(w.Hq):
        g = h // w.G
        logits = (K[g] @ w.q[0, h].double()) / math.sqrt(128)
        want = torch.softmax(logits, 0) @ V[g]
        assert np.abs(r.out[0, h] - want.numpy()).max() < 1e-12
        assert abs(r.lse[0, h] - float(torch.logsumexp(logits, 0))) < 1e-12


def test_permuting_middle_blocks_permutes_mask_and_keeps_output(oracle):
    w = make_workload("C1", N=4096)
    nb = w.num_blocks(0)
    codes, scales = oracle.quantize(w.bits("k_cache"), None, w.seq_lens, w.max_blocks)
    r = _decode(oracle, w, codes, scales, 6.0)
    perm = np.arange(nb)
    rng = np.random.default_rng(3)
    mid = np.arange(1, nb - 16)
    perm[mid] = rng.permutation(mid)
    w2 = make_workload("C1", N=4096)
    w2.k_cache = w.k_cache[perm].clone()
    w2.v_cache = w.v_cache[perm].clone()
    c2, s2 = oracle.quantize(w2.bits("k_cache"), None, w2.seq_lens, w2.max_blocks)
    r2 = _decode(oracle, w2, c2, s2, 6.0)
    assert np.array_equal(r2.kept[0, :, :nb], r.kept[0, :, :nb][:, perm])
    assert np.abs(r2.out - r.out).max() < 1e-12


def test_paged_equals_contiguous_and_poison_is_never_read(oracle):
    w = make_workload("C1", N=3000)
    wp = repage(w)
    c, s = oracle.quantize(w.bits("k_cache"), None, w.seq_lens, w.max_blocks)
    cp, sp = oracle.quantize(wp.bits("k_cache"), wp.block_table, wp.seq_lens, wp.max_blocks)
    r = _decode(oracle, w, c, s, 6.0)
    rp = _decode(oracle, wp, cp, sp, 6.0)
    assert np.array_equal(r.kept, rp.kept)
    assert np.array_equal(r.out, rp.out)
    assert np.abs(r.out).max() < 10.0


def test_scan_error_concentrates_as_the_theorem_says(oracle):
    """App. B theorem, used as a soft check: with sigma = s/2 per channel (half a quantization step) and
    alpha = |q|/sqrt(d), the frequency of |s_hat - s| >= lambda stays under 2 exp(-lambda^2 / (2 sigma^2 alpha^2))."""
    w = make_workload("C2", N=4096, sink=False)
    codes, scales = oracle.quantize(w.bits("k_cache"), None, w.seq_lens, w.max_blocks)
    K = bits_to_f64(w.bits("k_cache"))[:, 0].reshape(-1, 128)
    S = scales.view(np.float16).astype(np.float64)[:, 0]
    Khat = (CODEBOOK[codes[:, 0]] * S[:, None, :]).reshape(-1, 128)
    q = bits_to_f64(w.bits("q"))[0, 0]
    err = (Khat - K) @ q / math.sqrt(128)
    sigma = S.max() / 2
    alpha = np.linalg.norm(q) / math.sqrt(128)
    for lam in [1.0, 2.0, 3.0]:
        bound = 2 * math.exp(-lam ** 2 / (2 * sigma ** 2 * alpha ** 2))
        assert (np.abs(err) >= lam).mean() <= bound
    assert abs(err.mean()) < 0.2


def test_empty_sequence_and_argument_errors(oracle):
    w = make_workload("C1", N=256)
    codes, scales = oracle.quantize(w.bits("k_cache"), None, w.seq_lens, w.max_blocks)
    seq0 = np.array([0], dtype=np.int32)
    r = oracle.decode(w.bits("q"), w.bits("k_cache"), w.bits("v_cache"), codes, scales, None, seq0, w.max_blocks, 6.0)
    assert np.all(r.out == 0) and np.all(np.isneginf(r.lse))
    with pytest.raises(ValueError):
        _decode(oracle, w, codes, scales, -1.0)
    with pytest.raises(ValueError):
        _decode(oracle, w, codes, scales, float("nan"))
