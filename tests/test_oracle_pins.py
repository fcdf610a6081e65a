"""Pins for the CPU checker: every function is tied to something other than itself --
values the paper prints, closed forms, invariants, library routines or brute force."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as orc
from ocs_inputs import configs, prng

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append(line.split())
    return rows


# ----------------------------------------------------------------------------- Section 3.4
def test_split_count_is_ceil_rC():
    assert orc.num_splits(512, 0.05) == 26
    assert orc.num_splits(256, 0.02) == 6
    assert [orc.num_splits(25088, r) for r in (0, .01, .02, .05, .1)] == [0, 251, 502, 1255, 2509]
    assert orc.num_splits(650, 0.02) == 13          # 0.02*650 is 13 in exact arithmetic
    assert [orc.num_splits(c, .01) for c in (3, 64, 128, 256, 512, 1024, 2048)] == [1, 1, 2, 3, 6, 11, 21]
    for c in range(1, 300):
        for num in range(0, 40):
            r = num / 100.0
            assert orc.num_splits(c, r) == math.ceil(Fraction(num, 100) * c)


def test_resnet50_size_overhead_matches_table5():
    """Table 5: relative weight size of ResNet-50 at r = .01/.02/.05/.1 is 1.01/1.02/1.05/1.1;
    Section 5.2: r = 0.01 is a single split in many layers."""
    layers, fc = configs.resnet50_layers()
    alls = layers + [fc]
    base = sum(l.O * l.C * l.k * l.k for l in alls)
    for ratio, printed in _read_golden("table5_resnet50_weight_overhead.txt"):
        tot = sum(l.O * (l.C + orc.num_splits(l.C, float(ratio))) * l.k * l.k for l in alls)
        skip = sum(l.O * (l.C + (0 if l.name == "conv1" else orc.num_splits(l.C, float(ratio)))) * l.k * l.k
                   for l in alls)
        assert tot / base >= 1 + float(ratio)           # Section 5.4: r is a lower bound
        assert round(tot / base, len(printed.split(".")[1])) == float(printed)
        assert round(skip / base, len(printed.split(".")[1])) == float(printed)
    assert sum(1 for l in alls if orc.num_splits(l.C, 0.01) == 1) >= 4


# ----------------------------------------------------------------------------- Section 3.3
def _Q(x: Fraction) -> int:
    return math.floor(x + Fraction(1, 2))


def test_paper_worked_example_w3():
    """Section 3.3: w = 3 splits into 1.5 and 1.5, both rounded the same way, so the naive
    halves no longer sum to Q(w)."""
    W = np.array([[3.0]], dtype=np.float32)
    out, idx, order, _ = orc.split(W, 1, qa_step=0.0)
    assert out.tolist() == [[1.5, 1.5]] and idx.tolist() == [0, 0] and order.tolist() == [0]
    assert _Q(Fraction(1.5)) + _Q(Fraction(1.5)) == 4 != _Q(Fraction(3))
    qa, _, _, _ = orc.split(W, 1, qa_step=1.0)
    assert qa.tolist() == [[1.25, 1.75]]          # (w - .5)/2 stays in place, (w + .5)/2 is appended
    assert _Q(Fraction(1.25)) + _Q(Fraction(1.75)) == 3


def test_qa_identity_and_hermite_bruteforce():
    """Q((w-.5)/2) + Q((w+.5)/2) = Q(w) for Q = floor(x + 1/2) on a fine grid, evaluated exactly on
    what the checker's split produced; the naive rule fails somewhere; Hermite with n = 2."""
    ws = np.arange(-40 * 64, 40 * 64 + 1, dtype=np.float64) / 64.0
    # one column per value: a [1, n] matrix, one split each -> do them one at a time through
    # the checker so that each value is the channel maximum
    naive_fail = 0
    for chunk in np.array_split(ws, 64):
        for w in chunk[:: max(1, len(chunk) // 12)]:
            W = np.array([[w]], dtype=np.float32)
            qa, _, _, _ = orc.split(W, 1, qa_step=1.0)
            a, b = Fraction(float(qa[0, 0])), Fraction(float(qa[0, 1]))
            assert a == (Fraction(w) - Fraction(1, 2)) / 2 and b == (Fraction(w) + Fraction(1, 2)) / 2
            assert _Q(a) + _Q(b) == _Q(Fraction(w))
            nv, _, _, _ = orc.split(W, 1, qa_step=0.0)
            naive_fail += (_Q(Fraction(float(nv[0, 0]))) + _Q(Fraction(float(nv[0, 1]))) != _Q(Fraction(w)))
    assert naive_fail > 0
    for k in range(-40 * 64, 40 * 64 + 1):
        x = Fraction(k, 64)
        assert math.floor(x) + math.floor(x + Fraction(1, 2)) == math.floor(2 * x)
        assert _Q((x - Fraction(1, 2)) / 2) + _Q((x + Fraction(1, 2)) / 2) == _Q(x)


def test_qa_split_whole_channel_in_grid_units():
    """A whole channel moves together (Section 3.2) and every element gets the QA pair."""
    rng = np.random.default_rng(5)
    W = (rng.integers(-200, 200, size=(7, 5)) / 8.0).astype(np.float32)
    W[3, 2] = 50.0
    out, idx, order, mx = orc.split(W, 1, qa_step=1.0)
    assert order.tolist() == [2] and idx.tolist() == [0, 1, 2, 3, 4, 2]
    np.testing.assert_array_equal(out[:, [0, 1, 3, 4]], W[:, [0, 1, 3, 4]])
    np.testing.assert_array_equal(out[:, 2], (W[:, 2] - 0.5) / 2)
    np.testing.assert_array_equal(out[:, 5], (W[:, 2] + 0.5) / 2)
    assert mx == (50.0, max(25.25, float(np.abs(out).max())))


# ----------------------------------------------------------------------------- Eq. 3
@pytest.mark.parametrize("shape,S", [((33, 20), 7), ((16, 12, 3, 3), 5), ((9, 1), 4), ((5, 6), 0), ((4, 3), 9)])
def test_functional_identity_and_exact_halving(shape, S):
    rng = np.random.default_rng(11)
    W = rng.laplace(0, 0.02, size=shape).astype(np.float32)
    W.reshape(-1)[rng.integers(0, W.size, 3)] *= 30
    out, idx, order, mx = orc.split(W, S, qa_step=0.0, literal=True)
    Cn = shape[1]
    assert idx[:Cn].tolist() == list(range(Cn))
    # every entry is the source value times an exact power of two, per-source sums are exact
    src = W[:, idx]
    ratio = np.where(src != 0, out / np.where(src == 0, 1, src), 1.0)
    assert np.all(np.log2(ratio) == np.round(np.log2(ratio)))
    summed = np.zeros(W.shape, dtype=np.float64)
    np.add.at(summed, (slice(None), idx), out.astype(np.float64))   # exact: binary fractions of one value
    np.testing.assert_array_equal(summed, W.astype(np.float64))
    # layer output unchanged (Eq. 3 equals Eq. 2) for a random activation vector
    x = rng.standard_normal(Cn)
    W2 = W.reshape(shape[0], Cn, -1).astype(np.float64)
    o2 = out.reshape(shape[0], Cn + S, -1).astype(np.float64)
    y_ref = np.einsum("c,ocr->or", x, W2)
    y_new = np.einsum("c,ocr->or", x[idx], o2)
    np.testing.assert_allclose(y_new, y_ref, rtol=0, atol=1e-12 * np.abs(W2).sum())
    assert mx[0] == np.abs(W).max() and mx[1] == np.abs(out).max()


# ----------------------------------------------------------------------------- Eq. 4
def test_activation_ocs_keeps_the_layer_and_halves_the_outlier():
    """Eq. 4: with the chosen activation channels duplicated and halved and their weight columns
    duplicated unchanged, the layer output is the original one; on integer data every sum is exact."""
    rng = np.random.default_rng(23)
    M, Cn, N, S = 7, 12, 5, 6
    A = (rng.integers(-8, 9, size=(M, Cn)) * 64).astype(np.float32)      # halvings stay integers
    A[3, 4] = 64 * 40                                                      # the batch's outlier
    W = rng.integers(-9, 10, size=(N, Cn)).astype(np.int8)
    Ap, idx, order, mx = orc.act_ocs(A, S)
    Wd = orc.dup_weight_columns(W, idx)
    assert Wd.shape == (N, Cn + S) and np.array_equal(Wd[:, :Cn], W)
    for s in range(S):
        assert np.array_equal(Wd[:, Cn + s], W[:, idx[Cn + s]])
    y_ref = A.astype(np.int64) @ W.astype(np.int64).T
    y_new = Ap.astype(np.float64) @ Wd.astype(np.float64).T
    np.testing.assert_array_equal(y_new, y_ref.astype(np.float64))
    # both copies carry half of the value they were split from, the outlier's channel goes first
    assert order[0] == 4 and idx[Cn] == 4
    assert mx[0] == 64 * 40 and mx[1] < mx[0]
    cols = np.zeros((M, Cn), dtype=np.float64)
    np.add.at(cols, (slice(None), idx), Ap.astype(np.float64))
    np.testing.assert_array_equal(cols, A.astype(np.float64))
    # a channel split once: both copies are exactly a/2 (the plain split of Section 3.3)
    A1, idx1, _, _ = orc.act_ocs(A, 1)
    np.testing.assert_array_equal(A1[:, 4], A[:, 4] * 0.5)
    np.testing.assert_array_equal(A1[:, Cn], A[:, 4] * 0.5)
    others = [c for c in range(Cn) if c != 4]
    np.testing.assert_array_equal(A1[:, others], A[:, others])


def test_activation_ocs_layer_is_the_expanded_integer_layer():
    """The composed layer against a plain integer matmul on its own outputs, and the grid refinement
    the split buys: the expanded batch's max |a'| is what sets the scale."""
    c1 = configs.config1()
    A = c1["A"].copy()
    A[2, 17] = 25.0
    Wc, w_scale = orc.quantize(c1["W"], 8, True, orc.maxabs(c1["W"]))
    S = 5
    Y, acc, ac, a_scale, idx = orc.act_ocs_linear(A, S, 6, False, Wc, w_scale, None)
    ref = ac.astype(np.int64) @ Wc[:, idx].astype(np.int64).T
    np.testing.assert_array_equal(acc, ref)
    _, a_scale0 = orc.quantize(A, 6, False, orc.maxabs(A))
    assert a_scale < a_scale0 and idx[A.shape[1]] == 17
    assert ac.max() == 63 and ac.min() >= 0


# ----------------------------------------------------------------------------- Section 5.3
@pytest.mark.parametrize("rows,Cn,S,q,seed", [(50, 16, 4, 0.99, 0), (7, 5, 5, 0.5, 1), (200, 33, 1, 0.9, 2),
                                               (3, 4, 0, 0.99, 3), (64, 8, 3, 1.0, 4)])
def test_static_channel_choice_against_library_routines(rows, Cn, S, q, seed):
    """Threshold = numpy's nearest-rank quantile of |a|; counts and the top-S rule recomputed with
    library routines (stable argsort on negated counts = highest count first, ties by index)."""
    rng = np.random.default_rng(seed)
    P = rng.standard_normal((rows, Cn)).astype(np.float32)
    P[:, Cn // 2] *= 3.0                                  # one channel with heavier tails
    P[rng.integers(0, rows, 5), rng.integers(0, Cn, 5)] = 0.0
    sel, counts, thr = orc.act_select(P, S, q)
    ref_thr = np.quantile(np.abs(P).ravel(), q, method="inverted_cdf")
    assert np.float32(thr) == np.float32(ref_thr)
    ref_counts = (np.abs(P) > ref_thr).sum(axis=0)
    np.testing.assert_array_equal(counts, ref_counts)
    assert counts.sum() == P.size - np.sum(np.abs(P).ravel() <= ref_thr)
    np.testing.assert_array_equal(sel, np.argsort(-ref_counts, kind="stable")[:S])
    if S and q < 1.0:
        assert Cn // 2 in sel.tolist()


def test_static_channel_choice_tiny_worked_case():
    """Ten samples of three channels, by hand: 0.9-quantile of |a| is the 27th smallest of 30."""
    P = np.zeros((10, 3), np.float32)
    P[:, 0] = np.arange(1, 11)            # 1..10
    P[:, 1] = -np.arange(11, 21)          # -11..-20: the largest magnitudes
    P[:, 2] = np.arange(21, 31) * 0.01    # small
    sel, counts, thr = orc.act_select(P, 2, 0.9)
    assert thr == 17.0 and counts.tolist() == [0, 3, 0]
    assert sel.tolist() == [1, 0]         # the tie between channels 0 and 2 goes to the smaller index


def test_static_activation_split_is_eq4_with_a_fixed_list():
    rng = np.random.default_rng(5)
    M, Cn, N = 9, 10, 4
    A = (rng.integers(-20, 21, size=(M, Cn)) * 2).astype(np.float32)
    W = rng.integers(-9, 10, size=(N, Cn)).astype(np.int8)
    sel = np.array([7, 2, 3], np.int32)
    Ap, idx = orc.act_split_static(A, sel)
    assert idx.tolist() == list(range(Cn)) + [7, 2, 3]
    for s, c in enumerate(sel):
        np.testing.assert_array_equal(Ap[:, c], A[:, c] / 2)
        np.testing.assert_array_equal(Ap[:, Cn + s], A[:, c] / 2)
    rest = [c for c in range(Cn) if c not in sel.tolist()]
    np.testing.assert_array_equal(Ap[:, rest], A[:, rest])
    Wd = orc.dup_weight_columns(W, idx)
    np.testing.assert_array_equal(Ap.astype(np.float64) @ Wd.astype(np.float64).T,
                                  (A.astype(np.int64) @ W.astype(np.int64).T).astype(np.float64))
    # the same list applied through the greedy per-batch rule when that rule picks these channels once each
    B = np.ones((2, 4), np.float32)
    B[0, 3], B[1, 1] = 9.0, 8.0
    Bp, bidx, order, _ = orc.act_ocs(B, 2)
    Bs, sidx = orc.act_split_static(B, order)
    np.testing.assert_array_equal(Bp, Bs)
    np.testing.assert_array_equal(bidx, sidx)
    with pytest.raises(RuntimeError):
        orc.act_split_static(A, np.array([1, 1], np.int32))        # a channel listed twice
    with pytest.raises(RuntimeError):
        orc.act_split_static(A, np.array([Cn], np.int32))


def test_activation_ocs_lowers_the_layer_error_on_outlier_batches():
    """Direction of Table 4 (6 activation bits, r = 0.02): on a batch with a few outlier channels the layer
    output after per-batch activation OCS is closer to the float layer than without it, and a static choice
    made on a profile batch with the same outlier channels does as well."""
    rng = np.random.default_rng(29)
    M, Cn, N = 64, 256, 32
    A = np.abs(rng.standard_normal((M, Cn))).astype(np.float32)
    hot = [17, 101, 200]
    A[:, hot] *= 12.0
    P = np.abs(rng.standard_normal((512, Cn))).astype(np.float32)
    P[:, hot] *= 12.0
    W = rng.laplace(0, 0.02, size=(N, Cn)).astype(np.float32)
    Wc, ws = orc.quantize(W, 8, True, orc.maxabs(W))
    y_ref = A.astype(np.float64) @ (Wc.astype(np.float64) * ws).T
    S = orc.num_splits(Cn, 0.02)

    def err(Y):
        return float(np.mean((Y.astype(np.float64) - y_ref) ** 2))

    ac0, as0 = orc.quantize(A, 6, False, orc.maxabs(A))
    e_plain = err(orc.qlinear(ac0, False, as0, Wc, ws, np.arange(Cn, dtype=np.int32))[0])
    e_batch = err(orc.act_ocs_linear(A, S, 6, False, Wc, ws)[0])
    sel, counts, _ = orc.act_select(P, S, 0.99)
    assert set(hot) <= set(sel.tolist())
    Ap, idx = orc.act_split_static(A, sel)
    acs, ass = orc.quantize(Ap, 6, False, orc.maxabs(Ap))
    e_static = err(orc.qlinear(acs, False, ass, orc.dup_weight_columns(Wc, idx), ws,
                               np.arange(Cn + S, dtype=np.int32))[0])
    assert e_batch < 0.6 * e_plain
    assert e_static < 0.6 * e_plain


def test_greedy_is_monotone_and_targets_the_outlier():
    """Section 3.4 / 5.2: each split halves the current maximum's channel; the maximum never
    rises; with a unique largest outlier the first split strictly narrows the range."""
    c1 = configs.config1()
    W = c1["W"]
    prev = np.abs(W).max()
    j0 = int(np.unravel_index(np.abs(W).argmax(), W.shape)[1])
    for S in range(1, 27):
        out, idx, order, mx = orc.split(W, S)
        cur = np.abs(out).max()
        assert cur <= prev
        prev = cur
        if S == 1:
            assert order[0] == j0 and cur < np.abs(W).max()
            assert np.abs(out[:, j0]).max() == np.abs(W[:, j0]).max() / 2
    # literal rescans and cached maxima agree, naive and QA
    for qa in (0.0, float(np.abs(W).max()) / 127):
        a = orc.split(W, 26, qa, literal=True)
        b = orc.split(W, 26, qa, literal=False)
        np.testing.assert_array_equal(a[0], b[0])
        np.testing.assert_array_equal(a[1], b[1])
        np.testing.assert_array_equal(a[2], b[2])
    # config 1 re-splits at least one copy (an appended index appears in split_order)
    assert (orc.split(W, 26)[2] >= 512).any()


def test_greedy_bruteforce_python():
    """Independent re-derivation of the greedy loop with python floats on a tiny tensor, ties
    included (equal magnitudes: smallest current index first)."""
    W = np.array([[4, -4, 1, 0.5], [1, 2, -4, 0.25]], dtype=np.float32)
    S = 6
    cols = [list(map(float, W[:, j])) for j in range(4)]
    src = [0, 1, 2, 3]
    order = []
    for _ in range(S):
        mags = [max(abs(v) for v in c) for c in cols]
        j = max(range(len(cols)), key=lambda t: (mags[t], -t))
        order.append(j)
        half = [v / 2 for v in cols[j]]
        cols[j] = half
        cols.append(list(half))
        src.append(src[j])
    out, idx, so, _ = orc.split(W, S, literal=True)
    assert so.tolist() == order and idx.tolist() == src
    np.testing.assert_array_equal(out, np.array(cols, dtype=np.float32).T)


def test_split_degenerate():
    Z = np.zeros((3, 4), dtype=np.float32)
    out, idx, order, mx = orc.split(Z, 5)
    assert not out.any() and order.tolist() == [0] * 5 and idx.tolist() == [0, 1, 2, 3, 0, 0, 0, 0, 0]
    W = np.array([[2.0], [-6.0]], dtype=np.float32)            # C = 1, S > C
    out, idx, order, mx = orc.split(W, 3)
    assert idx.tolist() == [0, 0, 0, 0] and order.tolist() == [0, 0, 1]
    np.testing.assert_array_equal(out, np.array([[.5, .5, .5, .5], [-1.5, -1.5, -1.5, -1.5]], dtype=np.float32))
    np.testing.assert_array_equal(out.sum(axis=1), W[:, 0])


# ----------------------------------------------------------------------------- Eq. 1
@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 8])
def test_linear_quant_grid(bits):
    """Eq. 1: 2^k - 1 grid points spanning [-max, max]; error at most half an increment."""
    rng = np.random.default_rng(bits)
    x = rng.uniform(-1, 1, 10000).astype(np.float32)
    x = np.concatenate([x, -x])
    alpha = orc.maxabs(x)
    assert alpha == np.abs(x).max()
    codes, scale = orc.quantize(x, bits, True, alpha)
    L = 2 ** (bits - 1) - 1
    assert codes.min() >= -L and codes.max() <= L
    assert len(np.unique(codes)) <= 2 ** bits - 1
    if bits <= 6:
        assert len(np.unique(codes)) == 2 ** bits - 1
    assert scale == np.float32(alpha) / np.float32(L)
    err = np.abs(x.astype(np.float64) - codes.astype(np.float64) * scale)
    assert err.max() <= 0.5 * scale * (1 + 1e-5)
    # textbook form round(x L / max) * max / L, in double, away from rounding ties
    t = x.astype(np.float64) * L / float(alpha)
    safe = np.abs(t - np.floor(t) - 0.5) > 1e-4
    assert np.array_equal(codes[safe], np.rint(t[safe]).astype(np.int8))
    assert codes[np.abs(x).argmax()] in (-L, L)


def test_quantize_clip_saturates_and_rne():
    x = np.array([-3.0, -1.0, -0.5, 0.0, 0.5, 1.0, 1.5, 2.5, 3.0, 100.0], dtype=np.float32)
    codes, scale = orc.quantize(x, 3, True, 3.0)               # L = 3, step 1
    assert scale == 1.0
    assert codes.tolist() == [-3, -1, 0, 0, 0, 1, 2, 2, 3, 3]     # halves to even, 100 saturates
    ucodes, uscale = orc.quantize(x, 2, False, 3.0)            # L_u = 3
    assert ucodes.dtype == np.uint8 and ucodes.tolist() == [0, 0, 0, 0, 0, 1, 2, 2, 3, 3]
    z, s = orc.quantize(np.zeros(5, np.float32), 8, True, 0.0)
    assert not z.any() and s == 0.0


# ----------------------------------------------------------------------------- Section 4.1
def _brute_clip(values, counts, m: Fraction, bits, n_cand, signed=True):
    """Exact rational evaluation of the histogram MSE for every candidate."""
    L = 2 ** (bits - 1) - 1 if signed else 2 ** bits - 1
    best, cbest, scores = None, None, []
    for c in range(1, n_cand + 1):
        alpha = Fraction(float(np.float32(float(m * c / n_cand))))   # thresholds are fp32 values
        assert abs(alpha - m * c / n_cand) <= m * Fraction(1, 2 ** 23)  # evenly spaced on (0, max]
        step = alpha / L
        sc = Fraction(0)
        for xb, h in zip(values, counts):
            t = xb / step
            q = math.floor(t + Fraction(1, 2))
            if t + Fraction(1, 2) == q and q % 2 == 1:   # exact tie: to even
                q -= 1
            q = max(-L if signed else 0, min(L, q))
            sc += h * (xb - q * step) ** 2
        scores.append(sc)
        if best is None or sc <= best:
            best, cbest = sc, c
    return cbest, scores


@pytest.mark.parametrize("bits,n_cand,seed", [(2, 8, 0), (3, 16, 1), (4, 16, 2), (3, 5, 3), (2, 16, 4)])
def test_clip_mse_bruteforce(bits, n_cand, seed):
    """Tiny tensors whose values sit on bin centres: the histogram is the data, so the search
    must agree with an exact enumeration of every (threshold, grid point)."""
    B = 64
    rng = np.random.default_rng(seed)
    m = 2.0                                         # power of two: bin edges exact in fp32
    bins = np.unique(np.concatenate([rng.integers(0, 20, 40), rng.integers(0, B - 1, 6), [B - 1]]))
    counts = rng.integers(1, 9, size=bins.size)
    vals = []
    for b, h in zip(bins, counts):
        centre = (b + 0.5) * m / B
        vals += [centre] * int(h)
    vals = np.array(vals, dtype=np.float32)
    vals[-1] = m                                    # the maximum itself falls in the last bin
    vals *= rng.choice([-1.0, 1.0], size=vals.size).astype(np.float32)
    res = orc.clip_mse(vals, bits, True, n_bins=B, n_candidates=n_cand)
    hist = res["hist"]
    assert hist.sum() == vals.size and res["max_abs"] == m
    expect = np.zeros(B, dtype=np.uint64)
    expect[bins] = counts.astype(np.uint64)
    np.testing.assert_array_equal(hist, expect)
    centres = [Fraction(int(b) * 2 + 1, 2) * Fraction(2, B) for b in range(B)]
    cbest, scores = _brute_clip(centres, [int(h) for h in hist], Fraction(2), bits, n_cand)
    np.testing.assert_allclose(res["scores"], [float(s) for s in scores], rtol=1e-12, atol=1e-15)
    gaps = sorted(float(s) for s in scores)
    if gaps[1] - gaps[0] > 1e-9:                    # unambiguous minimum
        assert res["alpha"] == np.float32(2.0 * cbest / n_cand)


def test_clip_mse_properties():
    rng = np.random.default_rng(7)
    x = rng.laplace(0, 0.01, 50000).astype(np.float32)
    x[17] = 1.0                                     # one huge outlier, few bits -> must clip
    r = orc.clip_mse(x, 3, True)
    assert 0 < r["alpha"] < 1.0
    assert r["hist"].sum() == x.size
    # candidates are evenly spaced on (0, max]; the last one is "no clipping"
    r8 = orc.clip_mse(x, 8, True, n_candidates=4)
    assert r8["alpha"] in [np.float32(0.25 * k) for k in (1, 2, 3, 4)]
    # the same search on the raw elements picks a nearby candidate
    ex = orc.clip_mse_exact(x[:5000], 4, True, 64)
    hs = orc.clip_mse(x[:5000], 4, True, 2048, 64)
    assert abs(ex["alpha"] - hs["alpha"]) <= 2 * orc.maxabs(x[:5000]) / 64 + 1e-9
    # scoring really is sum h * (x - Q(x))^2 at the bin centres: recompute with numpy
    m, B, L = r["max_abs"], 2048, 3
    centres = (np.arange(B) + 0.5) * (m / B)
    for c in (1, 37, 128):
        step = float(np.float32(m * c / 128)) / L
        q = np.clip(np.rint(centres / step), -L, L)
        np.testing.assert_allclose(r["scores"][c - 1], (r["hist"] * (centres - q * step) ** 2).sum(), rtol=1e-10)
    assert orc.clip_mse(np.zeros(10, np.float32), 4)["alpha"] == 0.0


def test_clip_none_is_last_candidate():
    """With every value on the 8-bit grid of its own maximum, no clipping has zero error and
    wins (ties go to the largest threshold)."""
    x = (np.arange(-127, 128) / 127.0).astype(np.float32)
    r = orc.clip_mse_exact(x, 8, True, 16)
    assert r["alpha"] == 1.0


# ----------------------------------------------------------------------------- Eq. 2 / 3 on codes
def test_qlinear_matches_expanded_and_folded_matmul():
    M, Cn, N, S = 9, 37, 13, 6
    A = configs.random_codes(1, 0, (M, Cn), 0, 255, np.uint8)
    Wc = configs.random_codes(1, 1, (N, Cn + S), -127, 127, np.int8)
    idx = np.concatenate([np.arange(Cn), configs.random_codes(1, 2, (S,), 0, Cn - 1, np.int32)]).astype(np.int32)
    bias = prng.normal(1, 9, (N,))
    Y, acc = orc.qlinear(A, False, 0.013, Wc, 0.0007, idx, bias)
    expanded = A.astype(np.int64)[:, idx] @ Wc.astype(np.int64).T
    np.testing.assert_array_equal(acc, expanded)
    folded = np.zeros((N, Cn), dtype=np.int64)
    np.add.at(folded, (slice(None), idx), Wc.astype(np.int64))
    np.testing.assert_array_equal(acc, A.astype(np.int64) @ folded.T)
    s = np.float32(0.013) * np.float32(0.0007)
    np.testing.assert_allclose(Y, acc.astype(np.float64) * float(s) + bias, rtol=2e-7, atol=1e-9)
    # signed activations, identity map = plain integer matmul
    As = configs.random_codes(2, 0, (M, Cn), -127, 127, np.int8)
    _, acc0 = orc.qlinear(As, True, 1.0, Wc[:, :Cn].copy(), 1.0, np.arange(Cn, dtype=np.int32))
    np.testing.assert_array_equal(acc0, As.astype(np.int64) @ Wc[:, :Cn].astype(np.int64).T)
    ms, ns = np.array([0, 3, 8], np.int32), np.array([12, 0, 5], np.int32)
    Ys, accs = orc.qlinear_samples(A, False, 0.013, Wc, 0.0007, idx, ms, ns, bias)
    np.testing.assert_array_equal(accs, acc[ms, ns])
    np.testing.assert_array_equal(Ys, Y[ms, ns])


def test_folded_codes_give_the_same_accumulators():
    """Folding against numpy's add.at, and the folded layer against the gathered one (Eq. 3 both ways)."""
    M, Cn, N, S = 9, 37, 13, 6
    A = configs.random_codes(3, 0, (M, Cn), 0, 255, np.uint8)
    Wc = configs.random_codes(3, 1, (N, Cn + S), -60, 60, np.int8)          # two or three copies still fit int8
    idx = np.concatenate([np.arange(Cn), [5, 5, 0, 36, 17, 5]]).astype(np.int32)
    Wc[:, [5, Cn, Cn + 1, Cn + 5]] //= 4                                      # channel 5 has four copies
    Wf, over = orc.fold_duplicates(Wc, idx, Cn)
    ref = np.zeros((N, Cn), dtype=np.int64)
    np.add.at(ref, (slice(None), idx), Wc.astype(np.int64))
    assert over == 0
    np.testing.assert_array_equal(Wf, ref)
    _, acc = orc.qlinear(A, False, 1.0, Wc, 1.0, idx)
    _, acc_f = orc.qlinear(A, False, 1.0, Wf, 1.0, np.arange(Cn, dtype=np.int32))
    np.testing.assert_array_equal(acc_f, acc)
    # conv weights: taps fold independently
    W4 = configs.random_codes(3, 2, (4, 6 + 2, 3, 3), -50, 50, np.int8)
    idx4 = np.array([0, 1, 2, 3, 4, 5, 2, 4], np.int32)
    W4f, over = orc.fold_duplicates(W4, idx4, 6)
    ref4 = W4[:, :6].astype(np.int64).copy()
    ref4[:, 2] += W4[:, 6]
    ref4[:, 4] += W4[:, 7]
    assert over == 0
    np.testing.assert_array_equal(W4f, ref4)
    # sums that leave int8 are counted and saturated
    big = np.full((1, 3), 100, np.int8)
    f, over = orc.fold_duplicates(big, np.array([0, 1, 0], np.int32), 2)
    assert over == 1 and f.tolist() == [[127, 100]]
    f, over = orc.fold_duplicates(-big, np.array([0, 1, 0], np.int32), 2)
    assert over == 1 and f.tolist() == [[-128, -100]]


@pytest.mark.parametrize("k,stride,pad,H", [(3, 1, 1, 7), (3, 2, 1, 8), (1, 2, 0, 6), (7, 2, 3, 11), (1, 1, 0, 5)])
def test_qconv_matches_library_conv(k, stride, pad, H):
    torch = pytest.importorskip("torch")
    Nb, Cn, O, S = 2, 5, 4, 3
    X = configs.random_codes(3, 0, (Nb, H, H + 1, Cn), 0, 255, np.uint8)
    Wc = configs.random_codes(3, 1, (O, Cn + S, k, k), -127, 127, np.int8)
    idx = np.concatenate([np.arange(Cn), [4, 0, 4]]).astype(np.int32)
    bias = prng.normal(3, 9, (O,))
    Y, acc = orc.qconv(X, False, 0.5, Wc, 0.25, idx, stride, pad, bias)
    xe = torch.from_numpy(X.astype(np.float64)[..., idx]).permute(0, 3, 1, 2)
    ref = torch.nn.functional.conv2d(xe, torch.from_numpy(Wc.astype(np.float64)), stride=stride, padding=pad)
    ref = ref.permute(0, 2, 3, 1).numpy()
    np.testing.assert_array_equal(acc, ref.astype(np.int64))
    np.testing.assert_allclose(Y, ref * 0.125 + bias, rtol=2e-7, atol=1e-9)


# ----------------------------------------------------------------------------- glue
def test_glue_against_library_routines():
    torch = pytest.importorskip("torch")
    x = prng.normal(5, 0, (2, 9, 11, 6))
    np.testing.assert_array_equal(orc.relu(x), np.maximum(x, 0))
    y = prng.normal(5, 1, (2, 9, 11, 6))
    np.testing.assert_array_equal(orc.add_relu(x, y, True), np.maximum(x + y, 0))
    np.testing.assert_array_equal(orc.add_relu(x, y, False), x + y)
    t = torch.from_numpy(x).permute(0, 3, 1, 2)
    mp = torch.nn.functional.max_pool2d(t, 3, 2, 1).permute(0, 2, 3, 1).numpy()
    np.testing.assert_array_equal(orc.maxpool3x3s2(x), mp)
    np.testing.assert_allclose(orc.global_avgpool(x), x.astype(np.float64).mean(axis=(1, 2)), rtol=1e-5, atol=1e-6)
    nchw = prng.normal(5, 2, (2, 3, 4, 5))
    np.testing.assert_array_equal(orc.nchw_to_nhwc(nchw), nchw.transpose(0, 2, 3, 1))


def test_lstm_cell_against_libm():
    xs = np.linspace(-30, 30, 2001)
    sg = np.array([orc.sigmoid(float(v)) for v in xs])
    th = np.array([orc.tanh(float(v)) for v in xs])
    np.testing.assert_allclose(sg, 1 / (1 + np.exp(-xs)), rtol=0, atol=3e-7)
    np.testing.assert_allclose(th, np.tanh(xs), rtol=0, atol=3e-7)
    assert orc.sigmoid(0.0) == 0.5 and orc.tanh(0.0) == 0.0
    b, hdim = 3, 5
    gi, gh = prng.normal(6, 0, (b, 4 * hdim)), prng.normal(6, 1, (b, 4 * hdim))
    c0 = prng.normal(6, 2, (b, hdim))
    c1, h1 = orc.lstm_cell(gi, gh, c0)
    z = (gi + gh).astype(np.float64)
    i, f, g, o = (z[:, k * hdim:(k + 1) * hdim] for k in range(4))
    sig = lambda v: 1 / (1 + np.exp(-v))
    c_ref = sig(f) * c0 + sig(i) * np.tanh(g)
    np.testing.assert_allclose(c1, c_ref, atol=2e-6)
    np.testing.assert_allclose(h1, sig(o) * np.tanh(c_ref), atol=2e-6)


# ----------------------------------------------------------------------------- inputs
def test_input_streams_are_reproducible_and_shaped():
    a, b = configs.config1(), configs.config1()
    np.testing.assert_array_equal(a["W"], b["W"])
    W = a["W"]
    std = 0.02 * np.sqrt(2)
    assert (np.abs(W) > 9.9 * std).sum() == 8 and np.abs(W).max() <= 20 * std * 1.0001
    assert a["A"].min() >= 0
    c3 = configs.config3(O=256, C=1568, M=8)
    big = np.abs(c3["W"]) == np.float32(15 * 0.005 * np.sqrt(2))
    assert big.sum() == round(1e-4 * 256 * 1568)
    u = prng.Stream(9, 0).uniform(0, 100000)
    assert abs(u.mean() - 0.5) < 5e-3 and 0 < u.min() and u.max() < 1
    np.testing.assert_array_equal(prng.Stream(9, 0).bits(1000, 10), prng.Stream(9, 0).bits(0, 1010)[1000:])


# ----------------------------------------------------------------------------- Section 4.1, element-wise scorer
@pytest.mark.parametrize("bits,n_cand,seed", [(2, 8, 0), (3, 16, 1), (4, 16, 2), (3, 5, 3), (4, 7, 4)])
def test_clip_mse_exact_bruteforce(bits, n_cand, seed):
    """The element-wise scorer against an exact rational enumeration of every (threshold, element):
    every element is its own 'bin' with count 1.  Values are small dyadic rationals, so the fp32
    inputs are exact and only the candidates' fp32 rounding enters (reproduced by _brute_clip)."""
    rng = np.random.default_rng(100 + seed)
    vals = (rng.integers(-64, 65, size=40) / 32.0).astype(np.float32)
    vals[7] = 2.0
    vals[11] = -1.96875
    m = Fraction(float(np.abs(vals).max()))
    res = orc.clip_mse_exact(vals, bits, True, n_cand)
    cbest, scores = _brute_clip([Fraction(float(v)) for v in vals], [1] * vals.size, m, bits, n_cand)
    np.testing.assert_allclose(res["scores"], [float(s) for s in scores], rtol=1e-12, atol=1e-15)
    gaps = sorted(float(s) for s in scores)
    if gaps[1] - gaps[0] > 1e-9:
        assert res["alpha"] == np.float32(float(m) * cbest / n_cand)
    # unsigned codes: non-negative data, grid {0..2^k - 1}
    uv = np.abs(vals)
    resu = orc.clip_mse_exact(uv, bits, False, n_cand)
    cb_u, sc_u = _brute_clip([Fraction(float(v)) for v in uv], [1] * uv.size, m, bits, n_cand, signed=False)
    np.testing.assert_allclose(resu["scores"], [float(s) for s in sc_u], rtol=1e-12, atol=1e-15)


# ----------------------------------------------------------------------------- Section 3.3, grid step of the QA split
def test_split_qa_two_pass_rule_in_grid_units():
    """Two-pass rule: the step is (max|W'| of a plain-halving run) / L.  The tensor is built so that this is
    exactly 1.0 for 4-bit codes (L = 7); the QA pair of every split element must then satisfy the identity of
    Section 3.3, Q((w - .5)/2) + Q((w + .5)/2) = Q(w) with Q = floor(x + 1/2), evaluated in exact rationals."""
    rng = np.random.default_rng(31)
    W = (rng.integers(-48, 49, size=(9, 12)) / 8.0).astype(np.float32)       # |w| <= 6
    W[2, 3], W[5, 7], W[0, 10] = 13.5, -12.25, 9.75                          # three outlier channels
    W[4, 1] = 7.0                                                            # the largest value left after 3 splits
    S = 3
    out, idx, order, mx, step = orc.split_qa(W, S, 4)
    plain, _, order0, mx0 = orc.split(W, S, 0.0)
    assert mx0[1] == 7.0 and step == 1.0                                     # predicted max / L
    assert order.tolist() == order0.tolist() == [3, 7, 10]
    ref, idx_r, order_r, mx_r = orc.split(W, S, 1.0)                          # same thing with the step given
    np.testing.assert_array_equal(out, ref)
    np.testing.assert_array_equal(idx, idx_r)
    assert mx == mx_r
    for s, ch in enumerate(order):
        for o in range(W.shape[0]):
            w, a, b = Fraction(float(W[o, ch])), Fraction(float(out[o, ch])), Fraction(float(out[o, 12 + s]))
            assert a == (w - Fraction(1, 2)) / 2 and b == (w + Fraction(1, 2)) / 2
            assert _Q(a) + _Q(b) == _Q(w)
    # S = 0: the step is max|W| / L
    _, _, _, mxz, stepz = orc.split_qa(W, 0, 4)
    assert stepz == np.float32(13.5) / np.float32(7)


# ----------------------------------------------------------------------------- Section 4.3 (KL)
def _brute_kl(hist, m, L, n_cand, eps=1e-4):
    """The divergence of every candidate, written out from the definition with exact integer level sums
    (python ints / Fractions for the ratios, math.log on the final ratio)."""
    B, n = len(hist), sum(hist)
    scores = []
    for c in range(1, n_cand + 1):
        alpha = Fraction(float(np.float32(float(m) * c / n_cand)))
        step = alpha / L
        nc = -(-c * B // n_cand)
        level = []
        for i in range(nc):
            t = Fraction(2 * i + 1, 2) * m / B / step
            q = math.floor(t + Fraction(1, 2))
            if t + Fraction(1, 2) == q and q % 2 == 1:
                q -= 1
            level.append(min(L, max(0, q)))
        kept = sum(hist[:nc])
        if kept == 0:
            scores.append(math.inf)
            continue
        clipped = n - kept
        P = [hist[i] + (clipped if i == nc - 1 else 0) for i in range(nc)]
        mass, nnz = {}, {}
        for i in range(nc):
            mass[level[i]] = mass.get(level[i], 0) + hist[i]
            nnz[level[i]] = nnz.get(level[i], 0) + (hist[i] > 0)
        smooth = hist[nc - 1] == 0 and clipped > 0
        kl = 0.0
        for i in range(nc):
            if P[i] == 0:
                continue
            p = Fraction(P[i], n)
            if hist[i] == 0:
                q = Fraction(eps)
            else:
                q = Fraction(mass[level[i]], nnz[level[i]] * kept)
                if smooth:
                    q = q * (1 - Fraction(eps))
            kl += float(p) * math.log(p / q)
        scores.append(kl)
    return scores


@pytest.mark.parametrize("bits,n_cand,B,seed", [(2, 8, 64, 0), (3, 16, 64, 1), (4, 16, 128, 2), (3, 5, 50, 3)])
def test_clip_kl_bruteforce(bits, n_cand, B, seed):
    rng = np.random.default_rng(200 + seed)
    m = 2.0
    counts = np.zeros(B, dtype=np.int64)
    pick = np.unique(np.concatenate([rng.integers(0, B // 3, 30), rng.integers(0, B - 1, 8), [B - 1]]))
    counts[pick] = rng.integers(1, 12, size=pick.size)
    vals = []
    for b in np.nonzero(counts)[0]:
        vals += [(b + 0.5) * m / B] * int(counts[b])
    vals = np.array(vals, dtype=np.float32)
    vals[-1] = m
    vals *= rng.choice([-1.0, 1.0], size=vals.size).astype(np.float32)
    res = orc.clip_kl(vals, bits, True, n_bins=B, n_candidates=n_cand)
    np.testing.assert_array_equal(res["hist"], counts.astype(np.uint64))
    L = 2 ** (bits - 1) - 1
    ref = _brute_kl([int(x) for x in counts], Fraction(2), L, n_cand)
    np.testing.assert_allclose(res["scores"], ref, rtol=1e-11, atol=1e-14)
    assert all(s >= -1e-15 for s in res["scores"])                       # a divergence
    order = np.argsort(ref, kind="stable")
    if ref[order[1]] - ref[order[0]] > 1e-9:
        assert res["alpha"] == np.float32(2.0 * (order[0] + 1) / n_cand)
    # the library's generic divergence routine on the same two distributions (one candidate, no empty last bin)
    scipy_stats = pytest.importorskip("scipy.stats")
    c = n_cand
    P = counts.astype(np.float64)
    lvl = np.clip(np.rint((np.arange(B) + 0.5) * (m / B) / (float(np.float32(m)) / L)), 0, L).astype(int)
    mass = np.bincount(lvl, weights=P, minlength=L + 1)
    nnz = np.bincount(lvl, weights=(P > 0).astype(float), minlength=L + 1)
    Q = np.where(P > 0, mass[lvl] / np.maximum(nnz[lvl], 1), 0.0)
    np.testing.assert_allclose(res["scores"][c - 1], scipy_stats.entropy(P, Q), rtol=1e-10, atol=1e-14)


def test_clip_kl_properties():
    # a tensor that already sits on the k-bit grid of its own maximum: quantizing it at the last candidate
    # changes nothing, so the divergence there is exactly zero and the last candidate wins
    for bits in (3, 4, 6):
        L = 2 ** (bits - 1) - 1
        rng = np.random.default_rng(bits)
        codes = np.concatenate([rng.integers(-L, L + 1, 4000), [L, -L]])
        x = (codes / L).astype(np.float32)
        r = orc.clip_kl(x, bits, True, 2048, 128)
        assert r["scores"][-1] == 0.0 and r["alpha"] == 1.0
        assert (r["scores"][:-1] > 0).all()
    # clipping is penalised through the mass that piles up in the last kept bin: with one far outlier
    # and few bits the search clips, with many bits on clean data it does not clip much
    rng = np.random.default_rng(9)
    x = rng.laplace(0, 0.01, 60000).astype(np.float32)
    x[5] = 1.0
    r3 = orc.clip_kl(x, 3, True)
    assert 0 < r3["alpha"] < 0.5
    # scale covariance: powers of two change nothing but the scale
    r3b = orc.clip_kl(x * np.float32(4.0), 3, True)
    assert r3b["alpha"] == np.float32(4.0) * np.float32(r3["alpha"])
    np.testing.assert_array_equal(r3b["scores"], r3["scores"])
    assert orc.clip_kl(np.zeros(10, np.float32), 4)["alpha"] == 0.0


# ----------------------------------------------------------------------------- Section 4.2 (ACIQ)
def test_aciq_multipliers_closed_forms():
    """The Laplace threshold is a Lambert-W value, the Gauss threshold the root of a monotone equation; both
    minimise the model error (clipping noise + step^2/12).  With 2^M grid intervals they are the constants
    the method's authors publish (Banner et al. 2018, the work Section 4.2 cites): 2.83 b, 3.89 b, 5.03 b and
    1.71 s, 2.15 s, 2.56 s for M = 2, 3, 4."""
    sp = pytest.importorskip("scipy.special")
    so = pytest.importorskip("scipy.optimize")
    ss = pytest.importorskip("scipy.stats")
    for M, lap, gau in ((2, 2.83, 1.71), (3, 3.89, 2.15), (4, 5.03, 2.56)):
        assert abs(orc.aciq_multiplier(2 ** M, True) - lap) < 0.01        # printed with two decimals
        assert abs(orc.aciq_multiplier(2 ** M, False) - gau) < 0.01
    for bits in range(2, 9):
        for L in (2 ** (bits - 1) - 1, 2 ** bits - 1):
            n_int = 2.0 * L
            t = orc.aciq_multiplier(n_int, True)
            assert abs(t - float(np.real(sp.lambertw(3 * n_int ** 2)))) < 1e-12 * t
            lap_err = lambda a: 2 * math.exp(-a) + (2 * a / n_int) ** 2 / 12            # b = 1
            opt = so.minimize_scalar(lap_err, bounds=(1e-3, 60), method="bounded", options=dict(xatol=1e-10))
            assert abs(opt.x - t) < 1e-5 * t
            g = orc.aciq_multiplier(n_int, False)
            gau_err = lambda a: 2 * ((1 + a * a) * ss.norm.sf(a) - a * ss.norm.pdf(a)) + (2 * a / n_int) ** 2 / 12
            optg = so.minimize_scalar(gau_err, bounds=(1e-3, 40), method="bounded", options=dict(xatol=1e-10))
            assert abs(optg.x - g) < 1e-5 * g
            # and the clipping-noise closed forms themselves, against numerical integration of (x - a)^2 f(x)
            si = pytest.importorskip("scipy.integrate")
            a = 1.7
            num = 2 * si.quad(lambda x: (x - a) ** 2 * ss.norm.pdf(x), a, np.inf)[0]
            assert abs(num - 2 * ((1 + a * a) * ss.norm.sf(a) - a * ss.norm.pdf(a))) < 1e-10
            numl = 2 * si.quad(lambda x: (x - a) ** 2 * 0.5 * math.exp(-x), a, np.inf)[0]
            assert abs(numl - 2 * math.exp(-a)) < 1e-10


def test_clip_aciq_on_exact_laplace_and_gauss_samples():
    """Deterministic quantile samples of the two densities: the fit recovers the scale, the likelihood test
    picks the right density, alpha = multiplier * scale, and the measured quantization MSE of the sample at
    that alpha is within a few percent of the best MSE over a fine sweep of thresholds."""
    ss = pytest.importorskip("scipy.stats")
    n = 200001
    u = (np.arange(n) + 0.5) / n
    for name, sample, scale_true in (("laplace", ss.laplace.ppf(u, scale=0.02), 0.02), ("gauss", ss.norm.ppf(u, scale=0.05), 0.05)):
        x = sample.astype(np.float32)
        for bits in (3, 4, 6):
            L = 2 ** (bits - 1) - 1
            r = orc.clip_aciq(x, bits, True, 2048)
            assert r["laplace"] == (name == "laplace")
            scale = r["b"] if name == "laplace" else r["sigma"]
            assert abs(scale - scale_true) < 2e-3 * scale_true                   # histogram moments: bin-width error
            assert r["multiplier"] == orc.aciq_multiplier(2 * L, name == "laplace")
            expect = np.float32(r["multiplier"] * scale)
            assert r["alpha"] == min(expect, np.float32(r["max_abs"]))

            def mse(alpha):
                codes, step = orc.quantize(x, bits, True, float(alpha))
                return float(np.mean((x.astype(np.float64) - codes.astype(np.float64) * step) ** 2))
            sweep = [mse(a) for a in np.linspace(0.3, 2.0, 35) * r["alpha"]]
            assert mse(r["alpha"]) <= 1.10 * min(sweep)
    # the threshold never exceeds the largest value; all-zero input
    tiny = np.array([0.1, -0.1, 0.1, 0.1], np.float32)
    assert orc.clip_aciq(tiny, 8, True)["alpha"] == np.float32(0.1)
    assert orc.clip_aciq(np.zeros(8, np.float32), 4)["alpha"] == 0.0
    # unsigned codes on non-negative data use L_u = 2^k - 1
    xu = np.abs(ss.norm.ppf(u, scale=1.0)).astype(np.float32)
    ru = orc.clip_aciq(xu, 4, False, 2048)
    assert not ru["laplace"] and ru["multiplier"] == orc.aciq_multiplier(2 * 15, False)


# ----------------------------------------------------------------------------- Section 3.4 (knapsack)
def test_range_curve_follows_the_greedy_loop():
    rng = np.random.default_rng(41)
    for shape in ((8, 10), (6, 7, 3, 3)):
        W = rng.laplace(0, 0.02, size=shape).astype(np.float32)
        W.reshape(-1)[rng.integers(0, W.size, 4)] *= 25
        curve = orc.range_curve(W, 9)
        assert curve[0] == np.abs(W).max()
        for s in range(10):
            _, _, _, mx = orc.split(W, s, 0.0, literal=True)
            assert curve[s] == np.float32(mx[1])
        assert all(curve[s + 1] <= curve[s] for s in range(9))


def test_knapsack_is_optimal_against_exhaustive_search():
    import itertools
    rng = np.random.default_rng(43)
    for trial in range(6):
        n_layers = int(rng.integers(3, 7))
        curves, cost = [], []
        for l in range(n_layers):
            O, Cn, R = int(rng.integers(2, 6)) * 4, int(rng.integers(3, 7)), int(rng.choice([1, 9]))
            W = rng.laplace(0, 0.02, size=(O, Cn * R)).astype(np.float32).reshape(O, Cn, R)
            W.reshape(-1)[rng.integers(0, W.size, 2)] *= float(rng.uniform(3, 30))
            curves.append(orc.range_curve(W, int(rng.integers(1, 4))))
            cost.append(O * R)
        budget = int(sum(c * (len(cv) - 1) for c, cv in zip(cost, curves)) * rng.uniform(0.2, 0.7))
        S, total = orc.knapsack(curves, cost, budget)
        assert sum(int(s) * c for s, c in zip(S, cost)) <= budget
        assert all(0 <= s <= len(cv) - 1 for s, cv in zip(S, curves))
        rew = lambda l, s: (Fraction(float(curves[l][0])) - Fraction(float(curves[l][s]))) / Fraction(float(curves[l][0]))
        best = max(sum(rew(l, s) for l, s in enumerate(alloc))
                   for alloc in itertools.product(*[range(len(cv)) for cv in curves])
                   if sum(s * c for s, c in zip(alloc, cost)) <= budget)
        got = sum(rew(l, int(s)) for l, s in enumerate(S))
        assert abs(float(got - best)) < 1e-12 and abs(total - float(best)) < 1e-12
    # zero budget: nothing is split; a budget that pays for everything: every layer takes what still helps
    S0, t0 = orc.knapsack(curves, cost, 0)
    assert not S0.any() and t0 == 0.0
