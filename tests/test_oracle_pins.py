"""Pins for the CPU oracle: it is checked against things other than itself - library
routines (torch conv2d / max_pool2d in fp64, numpy matmul), closed forms, hand-computed
fixtures, the paper's invariants (Eq. 4 linearity, bias cancellation, RRM == dense at
every frame), the Table 1 complexity law and Table 4's printed ratios."""
import itertools
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as TF

import workloads as wl
from workloads.nets import LayerSpec
from oracle import rrm_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _spec(dtype, c_in, h, w, c_out, k, s, p, rng, kind="conv", **kw):
    sp = LayerSpec(kind, dtype, c_in, h, w, c_out, k, k, s, p, src=0, **kw)
    if dtype == "f32":
        sp.weight = rng.standard_normal((c_out, c_in, k, k)).astype(np.float32)
        sp.bias = rng.standard_normal(c_out).astype(np.float32)
    else:
        lo = -1 if dtype == "bin" else -127
        sp.weight = rng.integers(lo, -lo + 1, size=(c_out, c_in, k, k)).astype(np.int8)
        if dtype == "bin":
            sp.weight[sp.weight == 0] = 1
        sp.bias = rng.integers(-50, 51, size=c_out).astype(np.int32)
    return sp


# ------------------------------------------------------------------ dense definition
@pytest.mark.parametrize("k,s,p", [(1, 1, 0), (3, 1, 1), (3, 2, 1), (5, 1, 2), (5, 2, 0),
                                   (7, 2, 3), (11, 4, 0), (3, 1, 0), (2, 2, 1)])
@pytest.mark.parametrize("dtype", ["f32", "i8"])
def test_conv_matches_library_routine(k, s, p, dtype):
    rng = np.random.default_rng(k * 100 + s * 10 + p)
    c_in, c_out, h, w = 3, 4, 13, 11
    if h + 2 * p < k:
        pytest.skip("kernel larger than padded input")
    sp = _spec(dtype, c_in, h, w, c_out, k, s, p, rng)
    if dtype == "f32":
        X = rng.standard_normal((2, c_in, h, w)).astype(np.float32)
    else:
        X = rng.integers(0, 128, size=(2, c_in, h, w)).astype(np.int8)
    P = orc.projection(sp, X)
    ref = TF.conv2d(torch.from_numpy(X.astype(np.float64)), torch.from_numpy(sp.weight.astype(np.float64)),
                    torch.from_numpy(sp.bias.astype(np.float64)), stride=s, padding=p).numpy()
    if dtype == "f32":
        np.testing.assert_allclose(P, ref, rtol=1e-12, atol=1e-12)
    else:
        assert P.dtype == np.int64
        np.testing.assert_array_equal(P, np.rint(ref).astype(np.int64))


def test_conv_hand_computed_fixture():
    vals = {}
    for line in open(os.path.join(GOLDEN, "hand_conv.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *nums = line.split()
        vals[key] = np.array([int(v) for v in nums])
    sp = LayerSpec("conv", "i8", 1, 3, 3, 1, 2, 2, 1, 0, src=0)
    sp.weight = vals["filter"].reshape(1, 1, 2, 2).astype(np.int8)
    sp.bias = vals["bias"].astype(np.int32)
    X = vals["input"].reshape(1, 1, 3, 3)
    np.testing.assert_array_equal(orc.projection(sp, X).ravel(), vals["output"])
    sp.stride, sp.pad = 2, 1
    np.testing.assert_array_equal(orc.projection(sp, X).ravel(), vals["output_s2p1"])
    # the same numbers in the fp64 instantiation
    sp.dtype = "f32"
    sp.weight = sp.weight.astype(np.float32)
    sp.bias = sp.bias.astype(np.float32)
    np.testing.assert_array_equal(orc.projection(sp, X.astype(np.float32)).ravel(), vals["output_s2p1"])


def test_one_hot_filter_is_a_shift():
    """A filter that is 1 at tap (ky,kx) of channel c and 0 elsewhere copies the input
    shifted by (ky-p, kx-p): pins orientation (no flip), row/column order, channel order."""
    rng = np.random.default_rng(5)
    c_in, h, w, k, p = 3, 7, 9, 3, 1
    X = rng.integers(0, 100, size=(1, c_in, h, w))
    for c, ky, kx in [(0, 0, 2), (2, 2, 0), (1, 1, 1), (1, 0, 1)]:
        sp = LayerSpec("conv", "i8", c_in, h, w, 1, k, k, 1, p, src=0)
        sp.weight = np.zeros((1, c_in, k, k), dtype=np.int8)
        sp.weight[0, c, ky, kx] = 1
        sp.bias = np.zeros(1, dtype=np.int32)
        P = orc.projection(sp, X)[0, 0]
        padded = np.pad(X[0, c], p)
        np.testing.assert_array_equal(P, padded[ky:ky + h, kx:kx + w])


def test_1x1_conv_is_per_pixel_matmul_and_fc_is_matmul():
    rng = np.random.default_rng(6)
    sp = _spec("f32", 5, 4, 6, 7, 1, 1, 0, rng)
    X = rng.standard_normal((2, 5, 4, 6)).astype(np.float32)
    P = orc.projection(sp, X)
    Wm = sp.weight.reshape(7, 5).astype(np.float64)
    ref = np.einsum("oc,nchw->nohw", Wm, X.astype(np.float64)) + sp.bias.astype(np.float64).reshape(1, -1, 1, 1)
    np.testing.assert_allclose(P, ref, rtol=1e-13, atol=1e-13)
    # FC against numpy matmul, and FC == conv over a 1x1 map
    fc = _spec("i8", 40, 1, 1, 9, 1, 1, 0, rng, kind="fc")
    x = rng.integers(0, 128, size=(3, 40)).astype(np.int8)
    Pf = orc.projection(fc, x)
    ref = x.astype(np.int64) @ fc.weight.reshape(9, 40).astype(np.int64).T + fc.bias.astype(np.int64)
    np.testing.assert_array_equal(Pf.reshape(3, 9), ref)
    fc.kind = "conv"
    np.testing.assert_array_equal(orc.projection(fc, x.reshape(3, 40, 1, 1)), Pf)


def test_maxpool_matches_library_routine():
    rng = np.random.default_rng(7)
    X = rng.standard_normal((2, 3, 13, 13))
    for k, s, p in [(3, 2, 0), (3, 2, 1), (2, 2, 0)]:
        ref = TF.max_pool2d(torch.from_numpy(X), k, s, p).numpy()
        np.testing.assert_array_equal(orc.maxpool(X, k, s, p), ref)
        Xi = rng.integers(-1000, 1000, size=(2, 3, 13, 13)).astype(np.int64)
        refi = TF.max_pool2d(torch.from_numpy(Xi.astype(np.float64)), k, s, p).numpy().astype(np.int64)
        np.testing.assert_array_equal(orc.maxpool(Xi, k, s, p), refi)


def test_requant_hand_cases():
    # (P + 2^(s-1)) >> s with arithmetic shift: ties go towards +infinity; clamp to +-127
    P = np.array([0, 7, 8, 9, 23, 24, -7, -8, -9, -24, -25, 100000, -100000])
    want = np.array([0, 0, 1, 1, 1, 2, 0, 0, -1, -1, -2, 127, -127])
    np.testing.assert_array_equal(orc.requant(P, 4), want)
    np.testing.assert_array_equal(orc.requant(np.array([5, -200]), 0), np.array([5, -127]))
    sp = LayerSpec("conv", "i8", 1, 1, 1, 1, act="relu", shift=4, src=0)
    got = orc.nonlinearity(sp, np.array([[[[40]], [[-40]]]]), res=np.array([[[[-1]], [[5]]]]))
    # 40 -> 3 (40+8>>4), +(-1) = 2 ; -40 -> -2 (-32>>4), +5 = 3
    np.testing.assert_array_equal(got.ravel(), [2, 3])
    sp.act = "none"
    np.testing.assert_array_equal(orc.nonlinearity(sp, np.array([[[[-4000]]]])).ravel(), [-127])


def test_sign_takes_pool_first_and_threshold_inclusive():
    sp = LayerSpec("conv", "bin", 1, 3, 3, 1, act="sign", pool=(3, 2, 0), theta=5, src=0)
    P = np.array([[[[1, 2, 3], [4, 5, -6], [-7, -8, -9]]]])
    assert orc.nonlinearity(sp, P).ravel().tolist() == [1]        # max 5 >= theta 5
    sp.theta = 6
    assert orc.nonlinearity(sp, P).ravel().tolist() == [-1]


# ----------------------------------------------------------- the paper's invariants
@pytest.mark.parametrize("dtype", ["f32", "i8", "bin"])
@pytest.mark.parametrize("k,s,p", [(3, 1, 1), (5, 2, 2), (1, 2, 0), (4, 3, 1)])
def test_linearity_and_bias_cancellation(dtype, k, s, p):
    """Eq. 4: (F*I_t + b) - (F*I_{t-1} + b) == F*(I_t - I_{t-1}), with no bias term."""
    rng = np.random.default_rng(10 + k)
    sp = _spec(dtype, 4, 9, 10, 5, k, s, p, rng)
    if dtype == "f32":
        A, B = (rng.standard_normal((1, 4, 9, 10)).astype(np.float32) for _ in range(2))
    elif dtype == "i8":
        A, B = (rng.integers(0, 128, size=(1, 4, 9, 10)) for _ in range(2))
    else:
        A, B = (rng.integers(0, 2, size=(1, 4, 9, 10)) * 2 - 1 for _ in range(2))
    Pa, Pb = orc.projection(sp, A), orc.projection(sp, B)
    D = A.astype(np.float64) - B.astype(np.float64) if dtype == "f32" else A - B
    nobias = orc.projection(sp, D, with_bias=False)
    sparse = np.zeros_like(Pa)
    orc.delta_accumulate(sp, D, sparse)
    if dtype == "f32":
        scale = np.abs(Pa).max()
        assert np.abs((Pa - Pb) - nobias).max() <= 1e-12 * scale
        assert np.abs(sparse - nobias).max() <= 1e-12 * scale
    else:
        np.testing.assert_array_equal(Pa - Pb, nobias)
        np.testing.assert_array_equal(sparse, nobias)
    if dtype == "bin":
        assert set(np.unique(D)) <= {-2, 0, 2}     # remaining entries are all +-2
    # bias cancels: a different bias changes the projection by a constant only
    sp2 = _spec(dtype, 4, 9, 10, 5, k, s, p, np.random.default_rng(10 + k))
    sp2.bias = (sp2.bias * 0 + 3).astype(sp2.bias.dtype)
    np.testing.assert_allclose(orc.projection(sp2, A) - orc.projection(sp2, B), Pa - Pb, atol=1e-9)


def _seq_for(layers, frames, rng):
    s0 = layers[0]
    if s0.dtype == "f32":
        base = np.maximum(rng.standard_normal((1, s0.c_in, s0.h, s0.w)), 0).astype(np.float32)
    else:
        base = rng.integers(0, 128, size=(1, s0.c_in, s0.h, s0.w)).astype(np.int8)
    seq = [base]
    for _ in range(frames - 1):
        f = seq[-1].copy()
        y, x = int(rng.integers(0, s0.h - 4)), int(rng.integers(0, s0.w - 4))
        f[:, :, y:y + 4, x:x + 4] = base[:, :, :4, :4][:, :, ::-1, :].copy() if rng.random() < .3 else \
            (np.maximum(rng.standard_normal((1, s0.c_in, 4, 4)), 0).astype(np.float32) if s0.dtype == "f32"
             else rng.integers(0, 128, size=(1, s0.c_in, 4, 4)).astype(np.int8))
        seq.append(f)
    return seq


@pytest.mark.parametrize("net", ["alex_f32", "alex_i8", "resnet_i8", "xnor"])
def test_recurrence_equals_dense_at_every_frame(net):
    """The paper's central claim: the RRM feature maps equal a dense recompute of each
    frame.  Runs Algorithm 1 and the dense definition on small versions of the stacks."""
    rng = np.random.default_rng(42)
    if net == "alex_f32":
        layers = wl.alexnet_convs("f32", hw=67, scale=16)
    elif net == "alex_i8":
        layers = wl.alexnet_convs("i8", hw=67, scale=16)
    elif net == "resnet_i8":
        layers = wl.resnet18_convs(hw=64, scale=8)
    else:
        layers = wl.xnor_alexnet_convs(hw=67, scale=8)
    seq = _seq_for(layers, 5, rng)
    rec = orc.Recurrence(layers)
    for t, frame in enumerate(seq):
        tens_r, P_r = rec.step(frame)
        tens_d, P_d = orc.dense_forward(layers, frame)
        for l in range(len(layers)):
            if layers[l].dtype == "f32":
                assert np.abs(P_r[l] - P_d[l]).max() <= 1e-11 * max(1.0, np.abs(P_d[l]).max())
            else:
                np.testing.assert_array_equal(P_r[l], P_d[l])
        if layers[0].dtype != "f32":
            for a, b in zip(tens_r, tens_d):
                np.testing.assert_array_equal(a, b)
        if t > 0:
            assert rec.density()[0] < 0.2          # only the redrawn patch is non-zero


def test_zero_delta_and_full_delta_steps():
    layers = wl.single_conv_f32(c_in=4, c_out=6, hw=10)
    rng = np.random.default_rng(3)
    X = np.maximum(rng.standard_normal((1, 4, 10, 10)), 0).astype(np.float32)
    rec = orc.Recurrence(layers)
    _, P1 = rec.step(X)                                      # rho = 1 from the zero state
    np.testing.assert_allclose(P1[0], orc.projection(layers[0], X), rtol=1e-13, atol=1e-13)
    _, P2 = rec.step(X)                                      # rho = 0
    assert rec.nnz == [0] and rec.macs == [0]
    np.testing.assert_array_equal(P2[0], P1[0])


def test_mac_accounting_follows_table_1():
    rng = np.random.default_rng(8)
    fc = _spec("i8", 64, 1, 1, 24, 1, 1, 0, rng, kind="fc")
    D = np.zeros((1, 64), dtype=np.int64)
    D[0, [3, 10, 11, 40]] = [5, -2, 7, 1]
    P = np.zeros((1, 24), dtype=np.int64)
    assert orc.delta_accumulate(fc, D, P) == 4 * 24          # rho * C_in * C_out
    cv = _spec("i8", 3, 12, 12, 5, 3, 1, 1, rng)
    D = np.zeros((1, 3, 12, 12), dtype=np.int64)
    D[0, 1, 5, 6] = 4
    D[0, 2, 7, 2] = -9                                        # interior points: k*k*C_out each
    P = np.zeros((1, 5, 12, 12), dtype=np.int64)
    assert orc.delta_accumulate(cv, D, P) == 2 * 9 * 5
    D[:] = 0
    D[0, 0, 0, 0] = 1                                         # corner: only 4 of 9 taps land inside
    assert orc.delta_accumulate(cv, D, P) == 4 * 5


def _golden(name):
    vals = {}
    for line in open(os.path.join(GOLDEN, name)):
        if line.startswith("#") or not line.strip():
            continue
        key, *nums = line.split()
        vals[key] = np.array([int(v) for v in nums])
    return vals


@pytest.mark.parametrize("dtype", ["i8", "f32"])
def test_fc_delta_hand_computed_fixture(dtype):
    """FC branch of Algorithm 1's update on a 3 x 4 matrix whose rows, columns and streams all differ, so a
    transposed weight index, a swapped stream / input index or a dropped entry changes the result."""
    v = _golden("hand_fc_delta.txt")
    fc = LayerSpec("fc", dtype, 4, 1, 1, 3, src=0)
    fc.weight = v["weight"].reshape(3, 4, 1, 1).astype(np.float32 if dtype == "f32" else np.int8)
    fc.bias = np.zeros(3, dtype=np.float32 if dtype == "f32" else np.int32)
    dt = np.float64 if dtype == "f32" else np.int64
    P = v["p_prev"].reshape(2, 3).astype(dt)
    macs = orc.delta_accumulate(fc, v["delta"].reshape(2, 4).astype(dt), P)
    np.testing.assert_array_equal(P.ravel(), v["p_next"].astype(dt))
    assert macs == int(v["macs"][0])


@pytest.mark.parametrize("dtype", ["i8", "f32"])
def test_fc_delta_equals_matrix_product_of_the_delta(dtype):
    """Eq. 4 for the FC case: the column-by-column update onto zeros is W dI.  Checked against numpy's
    matmul (a library routine) and against the dense FC definition without bias, on a ragged c_in x c_out
    with several streams and mostly-zero deltas."""
    rng = np.random.default_rng(77)
    c_in, c_out, n = 37, 13, 3
    fc = _spec(dtype, c_in, 1, 1, c_out, 1, 1, 0, rng, kind="fc")
    dt = np.float64 if dtype == "f32" else np.int64
    D = np.zeros((n, c_in), dtype=dt)
    for s in range(n):
        idx = rng.choice(c_in, size=4 + 3 * s, replace=False)
        D[s, idx] = rng.standard_normal(idx.size) if dtype == "f32" else rng.integers(-254, 255, size=idx.size)
    P = np.zeros((n, c_out), dtype=dt)
    macs = orc.delta_accumulate(fc, D, P)
    Wm = fc.weight.reshape(c_out, c_in).astype(dt)
    ref = D @ Wm.T
    nobias = orc.projection(fc, D, with_bias=False).reshape(n, c_out)
    if dtype == "f32":
        np.testing.assert_allclose(P, ref, rtol=0, atol=1e-12 * np.abs(ref).max())
        np.testing.assert_allclose(P, nobias, rtol=0, atol=1e-12 * np.abs(ref).max())
    else:
        np.testing.assert_array_equal(P, ref)
        np.testing.assert_array_equal(P, nobias)
    assert macs == int(np.count_nonzero(D)) * c_out
    # an update onto a non-zero projection adds to it (Eq. 5), stream by stream
    P0 = (rng.standard_normal((n, c_out)) if dtype == "f32" else rng.integers(-1000, 1000, size=(n, c_out))).astype(dt)
    P1 = P0.copy()
    orc.delta_accumulate(fc, D, P1)
    if dtype == "f32":
        np.testing.assert_allclose(P1 - P0, ref, rtol=0, atol=1e-12 * np.abs(ref).max())
    else:
        np.testing.assert_array_equal(P1 - P0, ref)


@pytest.mark.parametrize("dtype", ["i8", "f32"])
def test_fc_recurrence_equals_dense_at_every_frame(dtype):
    """Algorithm 1 on a lone FC layer (and on an FC -> FC pair) against the dense definition, 5 frames."""
    rng = np.random.default_rng(12)
    c_in, c_mid, c_out, n = 48, 20, 9, 2
    a = _spec(dtype, c_in, 1, 1, c_mid, 1, 1, 0, rng, kind="fc", act="relu", shift=6 if dtype == "i8" else -1)
    b = _spec(dtype, c_mid, 1, 1, c_out, 1, 1, 0, rng, kind="fc")
    b.src = 1
    for layers in ([a], [a, b]):
        rec = orc.Recurrence(layers, n=n)
        x = (rng.standard_normal((n, c_in)).astype(np.float32) if dtype == "f32"
             else rng.integers(0, 128, size=(n, c_in)).astype(np.int8))
        for t in range(5):
            if t:
                j = rng.choice(c_in, size=5, replace=False)
                x = x.copy()
                x[:, j] = (rng.standard_normal((n, 5)).astype(np.float32) if dtype == "f32"
                           else rng.integers(0, 128, size=(n, 5)).astype(np.int8))
            tens_r, P_r = rec.step(x)
            tens_d, P_d = orc.dense_forward(layers, x)
            for l in range(len(layers)):
                if dtype == "f32":
                    assert np.abs(P_r[l] - P_d[l]).max() <= 1e-11 * max(1.0, np.abs(P_d[l]).max())
                else:
                    np.testing.assert_array_equal(P_r[l], P_d[l])
            if dtype != "f32":
                np.testing.assert_array_equal(tens_r[-1], tens_d[-1])
            if t:
                assert rec.nnz[0] <= 5 * n and rec.macs[0] == rec.nnz[0] * c_mid


def test_int32_accumulator_bound():
    # worst case of the largest contraction used here (fc6: 9216 inputs of magnitude <= 127)
    assert 9216 * 127 * 127 < 2 ** 31
    assert 384 * 9 * 2 < 2 ** 31                              # binary delta: |d| = 2, |w| = 1


def test_popcount_form_of_the_ternary_dot_product():
    """For binary inputs the non-zero deltas are +-2 (XNOR paragraph of the paper), so with
    `changed` = old^new, `new` the new sign bits and `B` the weight sign bits,
    sum(d*w) = 2*(popc(changed) - 2*popc(changed & (new ^ B))).  Brute force, 6 bits."""
    nb = 6
    for old, new, B in itertools.product(range(1 << nb), repeat=3):
        if (old * 7 + new * 3 + B) % 5:        # thin the 262144 cases deterministically
            continue
        bits = lambda v: np.array([(v >> i) & 1 for i in range(nb)]) * 2 - 1
        d = bits(new) - bits(old)
        assert set(np.unique(d)) <= {-2, 0, 2}
        want = int(np.dot(d, bits(B)))
        ch = old ^ new
        got = 2 * (bin(ch).count("1") - 2 * bin(ch & (new ^ B)).count("1"))
        assert got == want


def test_eta_reproduces_table_4():
    for line in open(os.path.join(GOLDEN, "table4_eta.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, _, S, S_rrm, eta_pct, tol = line.split()
        S, S_rrm, eta_pct, tol = float(S), float(S_rrm), float(eta_pct), float(tol)
        macs = np.array([3.0, 5.0, 11.0])                    # any MAC weights: densities are uniform
        eta = orc.speedup_ratio(np.full(3, 1 - S), np.full(3, 1 - S_rrm), macs)
        assert abs(eta * 100 - eta_pct) <= tol
        assert abs(orc.overall_sparsity(np.full(3, S), macs) - S) < 1e-12
    # Eq. 9 weights by MACs: a layer with 3x the MACs counts 3x
    assert abs(orc.overall_sparsity([0.0, 1.0], [1.0, 3.0]) - 0.75) < 1e-12
    assert abs(orc.speedup_ratio([1.0, 1.0], [0.5, 0.25], [1.0, 1.0]) - 2 / 0.75) < 1e-12


# -------------------------------------------------------------- workload sanity
def test_generated_stacks_are_not_degenerate():
    """The synthetic int8 / binary stacks must keep live activations (neither all zero
    nor all saturated), otherwise parity on deeper layers would be vacuous."""
    frame = wl.moving_rect_video(frames=1, hw=99, dtype="i8", seed=5)[0]
    for layers in (wl.alexnet_convs("i8", hw=99, scale=8), wl.xnor_alexnet_convs(hw=99, scale=8)):
        tens, _ = orc.dense_forward(layers, frame)
        for s, t in zip(layers, tens[1:]):
            if s.act == "sign":
                frac = float(np.mean(t > 0))
                assert 0.1 < frac < 0.9, (s.name, frac)
            elif s.shift >= 0:
                assert 0.1 < float(np.mean(t > 0)) and float(np.mean(np.abs(t) >= 127)) < 0.2, s.name


# ------------------------------------------------------------------ Sec. 3.4: truncation and Eq. 7 / Eq. 8
def _eps_video(frames=6, c=4, hw=10, seed=5, small=0.004, big=0.3):
    """Frames whose deltas are a mix of sub-threshold jitter (|d| <= small) and real changes (|d| ~ big)."""
    rng = np.random.default_rng(seed)
    v = np.empty((frames, 1, c, hw, hw), dtype=np.float32)
    v[0] = rng.random((1, c, hw, hw), dtype=np.float32)
    for t in range(1, frames):
        jitter = (rng.random((1, c, hw, hw), dtype=np.float32) - 0.5) * np.float32(2 * small)
        jitter[rng.random((1, c, hw, hw)) < 0.5] = 0
        v[t] = v[t - 1] + jitter
        v[t, 0, :, 2:5, 3:7] += np.float32(big) * rng.standard_normal((c, 3, 4)).astype(np.float32)
    return v


def test_truncated_recurrence_loses_exactly_the_filtered_truncated_part():
    """By linearity, P_eps(T) = dense(X_T) - F * (sum of the truncated parts): an independent route to the
    truncated recurrence's state (a dropped or doubly counted truncated entry breaks the equality)."""
    specs = wl.single_conv_f32(c_in=4, c_out=6, hw=10)
    v = _eps_video()
    eps = 0.01
    rec = orc.Recurrence(specs, eps=eps)
    U = np.zeros((1, 4, 10, 10))
    prev = np.zeros_like(v[0])
    l2 = 0.0
    for t in range(v.shape[0]):
        rec.step(v[t])
        d32 = v[t] - prev                                    # fp32 delta decides
        u = np.where(np.abs(d32) < np.float32(eps), v[t].astype(np.float64) - prev.astype(np.float64), 0.0)
        U += u
        l2 += float(np.sqrt((u * u).sum()))
        prev = v[t]
    want = orc.dense_forward(specs, v[-1])[1][0] - orc.projection(specs[0], U, with_bias=False)
    np.testing.assert_allclose(rec.P_prev[0], want, rtol=0, atol=1e-12)
    assert abs(rec.e_t - l2) <= 1e-12 * max(1.0, l2)
    assert rec.e_t > 0 and rec.macs[0] < orc.layer_macs(specs[0]) // 2      # the jitter was not multiplied


def test_truncation_hand_case_and_limits():
    s = wl.LayerSpec("conv", "f32", 1, 2, 2, 1, 1, 1, 1, 0, src=0)
    s.weight = np.full((1, 1, 1, 1), 2.0, dtype=np.float32)
    s.bias = np.array([1.0], dtype=np.float32)
    rec = orc.Recurrence([s], eps=0.01)
    x0 = np.zeros((1, 1, 2, 2), dtype=np.float32)
    rec.step(x0)
    x1 = np.array([0.005, 0.02, -0.003, 0.0], dtype=np.float32).reshape(1, 1, 2, 2)
    rec.step(x1)
    # kept: 0.02 -> P = 1 + 2 * 0.02 there; truncated: 0.005 and -0.003 -> l2 = sqrt(25e-6 + 9e-6)
    np.testing.assert_allclose(rec.P_prev[0].ravel(), [1.0, 1.0 + 2 * float(np.float32(0.02)), 1.0, 1.0], atol=1e-12)
    assert abs(rec.e_t - np.sqrt(float(np.float32(0.005)) ** 2 + float(np.float32(0.003)) ** 2)) < 1e-12
    assert rec.nnz[0] == 1
    # the snapshot moved on to x1: the same frame again has no delta at all, nothing more is truncated
    e = rec.e_t
    rec.step(x1)
    assert rec.nnz[0] == 0 and rec.e_t == e
    # a precise inference clears the accumulated value and the error
    _, projs = rec.reset_to(x1)
    assert rec.e_t == 0.0
    np.testing.assert_allclose(rec.P_prev[0], projs[0])
    # eps above every delta: nothing is ever multiplied, P stays at the bias
    big = orc.Recurrence([s], eps=10.0)
    big.step(x1)
    assert big.macs[0] == 0 and np.all(big.P_prev[0] == 1.0)
    # eps = 0 is the exact recurrence
    ex = orc.Recurrence([s], eps=0.0)
    ex.step(x1)
    np.testing.assert_allclose(ex.P_prev[0], orc.dense_forward([s], x1)[1][0], atol=1e-12)


def test_aecs_polynomial():
    mu = [0.5, -1.0, 2.0, 0.25, -0.125]
    for e in (0.0, 0.3, 2.0):
        assert abs(orc.aecs_predict(mu, e) - float(np.polyval(mu[::-1], e))) < 1e-12


def test_leaky_relu_matches_the_library_routine():
    import torch
    s = wl.LayerSpec("conv", "f32", 2, 5, 5, 3, 1, 1, 1, 0, act="leaky", src=0)
    P = np.random.default_rng(2).standard_normal((1, 3, 5, 5))
    got = orc.nonlinearity(s, P)
    want = torch.nn.functional.leaky_relu(torch.from_numpy(P), float(np.float32(0.1))).numpy()
    np.testing.assert_allclose(got, want, atol=1e-15)
    assert (got[P < 0] < 0).all() and (got[P > 0] == P[P > 0]).all()


# ------------------------------------------------------------------ explicit batch normalisation as part of f (Sec. 4.5)
def test_explicit_bn_hand_cases():
    # fp32: y = scale * P + shift per channel, then ReLU
    s = LayerSpec("conv", "f32", 1, 1, 2, 2, act="relu", src=0)
    s.bn_scale = np.array([2.0, -1.0], dtype=np.float32)
    s.bn_shift = np.array([0.5, 0.25], dtype=np.float32)
    P = np.array([[[[1.0, -3.0]], [[4.0, -2.0]]]])            # [1, 2 channels, 1, 2]
    # channel 0: 2*1+0.5 = 2.5, 2*(-3)+0.5 = -5.5 -> 0 ; channel 1: -4+0.25 = -3.75 -> 0, 2+0.25 = 2.25
    np.testing.assert_allclose(orc.nonlinearity(s, P).ravel(), [2.5, 0.0, 0.0, 2.25], atol=1e-15)
    # int8: q = clamp((P*m + a + 2^(s-1)) >> s, -127, 127), then + shortcut, then ReLU
    q = LayerSpec("conv", "i8", 1, 1, 1, 3, act="relu", shift=4, src=0)
    q.bn_scale = np.array([3, 1, 5], dtype=np.int32)
    q.bn_shift = np.array([-8, 7, 0], dtype=np.int32)
    P = np.array([[[[10]], [[-30]], [[1000]]]])
    # ch0: 30-8+8 = 30 >> 4 = 1 ; ch1: -30+7+8 = -15 >> 4 = -1 (arithmetic shift) ; ch2: 5000+8 >> 4 = 313 -> 127
    res = np.array([[[[0]], [[3]], [[-100]]]])
    # + shortcut: 1, 2, 27 ; ReLU keeps them
    np.testing.assert_array_equal(orc.nonlinearity(q, P, res=res).ravel(), [1, 2, 27])
    q.act = "none"
    np.testing.assert_array_equal(orc.nonlinearity(q, P).ravel(), [1, -1, 127])


def test_unfolded_bn_equals_the_folded_stack():
    """An affine after a linear layer folds into it: scale * (F*I + b) + shift = (scale F)*I + (scale b + shift).
    The oracle's unfolded stack must agree with its own evaluation of the folded one (in fp64; the folded
    filters are rounded to fp32, hence the tolerance), through ReLU and pooling, at every layer."""
    specs = wl.with_explicit_bn(wl.alexnet_convs("f32", hw=67, scale=16))
    folded = wl.fold_bn_f32(specs)
    assert all(f.bn_scale is None for f in folded) and all(s.bn_scale is not None for s in specs)
    frame = wl.moving_rect_video(frames=1, hw=67, dtype="f32", seed=5)[0]
    tu, _ = orc.dense_forward(specs, frame)
    tf, _ = orc.dense_forward(folded, frame)
    for a, b in zip(tu[1:], tf[1:]):
        assert np.abs(a - b).max() <= 1e-5 * max(1.0, np.abs(b).max())
    # and the affine really acts: without it the tensors differ
    plain = wl.alexnet_convs("f32", hw=67, scale=16)
    tp, _ = orc.dense_forward(plain, frame)
    assert np.abs(tp[1] - tu[1]).max() > 1e-3


@pytest.mark.parametrize("net", ["alex_f32", "resnet_i8"])
def test_recurrence_with_explicit_bn_equals_dense(net):
    rng = np.random.default_rng(7)
    layers = wl.with_explicit_bn(wl.alexnet_convs("f32", hw=67, scale=16) if net == "alex_f32" else wl.resnet18_convs(hw=64, scale=8))
    seq = _seq_for(layers, 4, rng)
    rec = orc.Recurrence(layers)
    for frame in seq:
        tens_r, P_r = rec.step(frame)
        tens_d, P_d = orc.dense_forward(layers, frame)
        for l in range(len(layers)):
            if layers[l].dtype == "f32":
                assert np.abs(P_r[l] - P_d[l]).max() <= 1e-11 * max(1.0, np.abs(P_d[l]).max())
            else:
                np.testing.assert_array_equal(P_r[l], P_d[l])
                np.testing.assert_array_equal(tens_r[l + 1], tens_d[l + 1])
    if net == "resnet_i8":       # the integer affine keeps the activations alive
        t = tens_d[-1]
        assert 0.05 < float(np.mean(t > 0)) and float(np.mean(np.abs(t) >= 127)) < 0.3
