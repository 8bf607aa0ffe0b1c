"""Approximate mode on the GPU (Sec. 3.4): delta entries below eps are truncated, the accumulated truncated
value e_t (Eq. 7) is kept on the device, a keyframe clears it.  Compared with the oracle's truncated recurrence:
at layer 0 both sides see the same fp32 inputs, so the truncation decisions and the counters agree exactly;
deeper layers see activations that differ in the last bits (fp32 vs fp64), so an entry within rounding of eps
can fall on the other side - the tolerance there allows for such rare flips (each moves P by at most eps * |w|)."""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import rrm_oracle as orc
from helpers import dev

pytestmark = pytest.mark.gpu


def _rrm():
    import paper_1802_09723_b200 as rrm
    return rrm


def _jitter_video(frames, c, hw, seed, small=0.004, big=0.3, n=1):
    rng = np.random.default_rng(seed)
    v = np.empty((frames, n, c, hw, hw), dtype=np.float32)
    v[0] = rng.random((n, c, hw, hw), dtype=np.float32)
    for t in range(1, frames):
        jitter = (rng.random((n, c, hw, hw), dtype=np.float32) - 0.5) * np.float32(2 * small)
        jitter[rng.random((n, c, hw, hw)) < 0.5] = 0
        v[t] = v[t - 1] + jitter
        y, x = int(rng.integers(0, hw - 6)), int(rng.integers(0, hw - 7))
        v[t, :, :, y:y + 5, x:x + 6] += np.float32(big) * rng.standard_normal((n, c, 5, 6)).astype(np.float32)
    return v


def test_single_layer_truncation_matches_the_oracle_every_frame():
    rrm = _rrm()
    specs = wl.single_conv_f32(c_in=16, c_out=24, hw=24)
    v = _jitter_video(8, 16, 24, seed=3, n=2)
    eps = 0.01
    net = rrm.net_from_specs(specs, n=2)
    net.set_epsilon(eps)
    rec = orc.Recurrence(specs, n=2, eps=eps)
    exact = orc.Recurrence(specs, n=2)
    out = net.new_output()
    for t in range(v.shape[0]):
        net.step(dev(v[t]), out)
        rec.step(v[t])
        exact.step(v[t])
        P = net.projection(0).cpu().numpy().astype(np.float64)
        scale = float(np.abs(rec.P_prev[0]).max())
        assert np.abs(P - rec.P_prev[0]).max() <= 1e-4 * scale, t
        st = net.stats(0)
        assert st["nnz_elems"] == rec.nnz[0] and st["active_macs"] == rec.macs[0], (t, st)
        e_t, per = net.truncation()
        assert abs(e_t - rec.e_t) <= 1e-5 * max(rec.e_t, 1e-9) and abs(per[0] - rec.trunc_l2[0]) <= 1e-5 * max(rec.trunc_l2[0], 1e-9)
    assert rec.e_t > 0 and rec.nnz[0] < exact.nnz[0] / 4                  # the jitter really was truncated
    assert np.abs(rec.P_prev[0] - exact.P_prev[0]).max() > 1e-6           # and the result really is approximate
    # a precise inference clears the accumulated value; the next frames accumulate from zero
    net.keyframe(dev(v[3]), out)
    rec.reset_to(v[3])
    assert net.truncation()[0] == 0.0
    net.step(dev(v[4]), out)
    rec.step(v[4])
    assert abs(net.truncation()[0] - rec.e_t) <= 1e-5 * max(rec.e_t, 1e-9)
    # eps = 0 again: exact from the next keyframe on
    net.set_epsilon(0.0)
    net.keyframe(dev(v[5]), out)
    net.step(dev(v[6]), out)
    want = orc.dense_forward(specs, v[6])[1][0]
    assert np.abs(net.projection(0).cpu().numpy() - want).max() <= 1e-4 * np.abs(want).max()
    net.close()


def test_small_fp32_stack_with_truncation():
    rrm = _rrm()
    specs = wl.alexnet_convs("f32", hw=99, scale=8)
    v = _jitter_video(6, 3, 99, seed=4, small=0.002, big=0.4)
    eps = 0.005
    net = rrm.net_from_specs(specs)
    net.set_epsilon(eps)
    rec = orc.Recurrence(specs, eps=eps)
    rec.reset_to(np.zeros_like(v[0]))                                      # the library's fresh state: exact response to a zero frame
    out = net.new_output()
    for t in range(v.shape[0]):
        net.step(dev(v[t]), out)
        rec.step(v[t])
        for l in range(len(specs)):
            P = net.projection(l).cpu().numpy().astype(np.float64)
            scale = float(np.abs(rec.P_prev[l]).max())
            assert np.abs(P - rec.P_prev[l]).max() <= 2e-4 * scale, (t, l)
        e_t, _ = net.truncation()
        assert abs(e_t - rec.e_t) <= 1e-4 * max(rec.e_t, 1e-9), (t, e_t, rec.e_t)
    net.close()


def test_epsilon_is_refused_for_integer_stacks_and_the_polynomial_is_horner():
    rrm = _rrm()
    net = rrm.net_from_specs(wl.alexnet_convs("i8", hw=99, scale=8))
    with pytest.raises(rrm.RRMError):
        net.set_epsilon(0.01)
    net.close()
    mu = [0.5, -1.0, 2.0, 0.25, -0.125]
    for e in (0.0, 0.3, 2.0):
        assert abs(rrm.aecs_predict(mu, e) - orc.aecs_predict(mu, e)) < 1e-12
