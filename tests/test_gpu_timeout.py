"""A bounded device-side wait that runs out is reported, not hung on, and leaves the context usable.

The only form in which this is run on a GPU: rrm_options.wait_limit = 0 on the two tensor-core kernels.  There
every role of a thread block (copy producers, filter loader, MMA issuer, epilogue) meets its first wait BEFORE it
has issued any asynchronous copy or MMA, so a wait that gives up at once lets the block leave with nothing in
flight: it frees its tensor memory and returns.  The host then reads bit 1 of rrm_stats.error_word and gets
RRM_ERR_TIMEOUT from rrm_get_stats.  After the limit is restored and the errors are cleared, a keyframe rebuilds
the state and the next frames match the CPU oracle again."""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import rrm_oracle as orc
from helpers import dev

pytestmark = pytest.mark.gpu

TIMEOUT_STATUS, TIMEOUT_BIT = -6, 2


def test_options_round_trip_and_validation():
    import paper_1802_09723_b200 as rrm
    layer = rrm.layer_from_spec(wl.fc6_i8(c_in=256, c_out=128)[0])
    o = layer.options()
    assert o["wait_limit"] == 1 << 20 and abs(o["stack_dense_activity"] - 0.75) < 1e-6 and o["stack_reprobe"] == 15
    assert o["layer_dense_activity"] > 1.0 and o["layer_delta_activity"] > 1.0            # the per-layer choice is opt-in
    layer.set_options(wait_limit=123, fc_dense_rows=0.5)
    o2 = layer.options()
    assert o2["wait_limit"] == 123 and abs(o2["fc_dense_rows"] - 0.5) < 1e-6 and o2["stack_reprobe"] == 15
    with pytest.raises(rrm.RRMError):
        layer.set_options(stack_reprobe=0)
    with pytest.raises(rrm.RRMError):
        layer.set_options(layer_dense_activity=0.2, layer_delta_activity=0.5)
    layer.close()


def test_few_row_fc_kernel_reports_a_wait_that_ran_out_and_recovers():
    import paper_1802_09723_b200 as rrm
    c_in, c_out, T = 1024, 512, 4
    spec = wl.fc6_i8(c_in=c_in, c_out=c_out)[0]
    seq = wl.fc_run_sequence(frames=T + 2, c_in=c_in, rho=0.05, seed=5)
    layer = rrm.layer_from_spec(spec)
    frames = dev(seq)
    Y = layer.new_output(frames=T)
    layer.dense_seq(frames[:T], Y, T)                         # healthy run first: the tensor-core kernel is the one in use
    for t in range(T):
        np.testing.assert_array_equal(Y[t].cpu().numpy().astype(np.int64), orc.dense_forward([spec], seq[t])[0][1])
    assert layer.stats(0)["error_word"] == 0
    layer.set_options(wait_limit=0)
    layer.dense_seq(frames[:T], Y, T)
    st = layer.stats(0, check=False)
    assert st["status"] == TIMEOUT_STATUS and st["error_word"] & TIMEOUT_BIT, st
    with pytest.raises(rrm.RRMError):
        layer.stats(0)
    # the context is intact: restore the limit, clear the flag, rebuild the state, step on
    layer.set_options(wait_limit=1 << 20)
    layer.clear_errors()
    layer.keyframe(frames[0], None)
    Y1 = layer.new_output()
    for t in range(1, T + 2):
        layer.step(frames[t], Y1)
        np.testing.assert_array_equal(Y1.cpu().numpy().astype(np.int64), orc.dense_forward([spec], seq[t])[0][1])
    assert layer.stats(0)["error_word"] == 0
    layer.close()


def test_tensor_core_conv_reports_a_wait_that_ran_out_and_recovers():
    import paper_1802_09723_b200 as rrm
    specs = wl.alexnet_convs("i8", hw=99, scale=8)
    video = wl.moving_rect_video(frames=4, hw=99, dtype="i8", seed=9, side=(12, 24))
    net = rrm.net_from_specs(specs, variant="tensor")
    out = net.new_output()
    net.step(dev(video[0]), out)
    assert net.stats(0)["error_word"] == 0 and net.stats(0)["variant"] == 2       # the tensor-core kernel runs these layers
    net.set_options(wait_limit=0)
    net.step(dev(video[1]), out)                               # the first layer's thread blocks give up at their first wait
    st = net.stats(0, check=False)
    assert st["status"] == TIMEOUT_STATUS and st["error_word"] & TIMEOUT_BIT, st
    net.set_options(wait_limit=1 << 20)
    net.clear_errors()
    net.keyframe(dev(video[1]), out)                           # a precise inference replaces the inconsistent state
    for t in (2, 3):
        net.step(dev(video[t]), out)
        _, P = orc.dense_forward(specs, video[t])
        for l in range(len(specs)):
            np.testing.assert_array_equal(net.projection(l).cpu().numpy().astype(np.int64), P[l])
    assert net.stats(0)["error_word"] == 0
    net.close()
