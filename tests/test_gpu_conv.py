"""GPU parity of the convolution path (single layers and layer stacks) against the CPU oracle.
Integer and binary layers must match bit for bit; fp32 layers within 1e-4 * max|P_dense| per
frame (the accumulated projection is compared at every frame, so drift would show)."""
import numpy as np
import pytest
import torch

import workloads as wl
from workloads.nets import LayerSpec, out_hw
from oracle import rrm_oracle as orc
from helpers import dev, pack_bits_nhwc, unpack_bits_nhwc

pytestmark = pytest.mark.gpu
F32_TOL = 1e-4


def _rrm():
    import paper_1802_09723_b200 as rrm
    return rrm


def _frame_to_dev(specs, frame):
    if specs[0].dtype == "bin":
        return dev(pack_bits_nhwc(frame).view(np.int32))
    return dev(frame)


def _out_kind(s):
    if s.dtype == "f32":
        return "f32"
    if s.act == "sign":
        return "bin"
    return "i8" if s.shift >= 0 else "i32"


def _compare(specs, net, frame, t, check_tensors=True):
    tens_d, P_d = orc.dense_forward(specs, frame)
    for l, s in enumerate(specs):
        P = net.projection(l).cpu().numpy()
        if s.dtype == "f32":
            scale = float(np.abs(P_d[l]).max())
            err = float(np.abs(P.astype(np.float64) - P_d[l]).max())
            assert err <= F32_TOL * scale, f"frame {t} layer {l} ({s.name}): err {err:.3e} scale {scale:.3e}"
        else:
            np.testing.assert_array_equal(P.astype(np.int64), P_d[l], err_msg=f"frame {t} layer {l} ({s.name})")
        if not check_tensors:
            continue
        T = net.tensor(l + 1).cpu().numpy()
        kind = _out_kind(s)
        if kind == "bin":
            np.testing.assert_array_equal(unpack_bits_nhwc(T.view(np.uint32), s.c_out), tens_d[l + 1],
                                          err_msg=f"frame {t} tensor {l + 1}")
        elif kind == "f32":
            scale = max(1e-30, float(np.abs(tens_d[l + 1]).max()))
            assert float(np.abs(T - tens_d[l + 1]).max()) <= F32_TOL * max(scale, float(np.abs(P_d[l]).max()))
        else:
            np.testing.assert_array_equal(T.astype(np.int64), tens_d[l + 1], err_msg=f"frame {t} tensor {l + 1}")


def _run(specs, video, n=1, check_frames=None, stats=False, keyframe_at=(), variant="auto", stats_frames=()):
    """stats: compare every frame's counters with the literal recurrence (small stacks).  stats_frames: the same at
    the named frames only, the recurrence being brought to the frame before by a dense pass (full-size stacks)."""
    rrm = _rrm()
    net = rrm.net_from_specs(specs, n=n, variant=variant)
    out = net.new_output()
    rec = orc.Recurrence(specs, n=n) if stats else None
    if rec is not None:
        # a fresh library state is the stack's response to the all-zero input pattern (all -1 for a
        # binary input); bring the literal recurrence to the same state
        rec.step(np.full_like(video[0], -1 if specs[0].dtype == "bin" else 0))
    for t in range(video.shape[0]):
        x = _frame_to_dev(specs, video[t])
        if t in keyframe_at:
            net.keyframe(x, out)
        else:
            net.step(x, out)
        if rec is not None:
            rec.step(video[t])
            if t not in keyframe_at:
                for l in range(len(specs)):
                    st = net.stats(l)
                    assert st["error_word"] == 0
                    if specs[0].dtype != "f32" or l == 0:
                        assert st["nnz_elems"] == rec.nnz[l], (t, l, st, rec.nnz[l])
                        assert st["active_macs"] == rec.macs[l], (t, l, st, rec.macs[l])
        if t in stats_frames:
            one = orc.Recurrence(specs, n=n)
            one.reset_to(video[t - 1])
            one.step(video[t])
            for l in range(len(specs)):
                st = net.stats(l)
                assert st["error_word"] == 0 and st["nnz_elems"] != -1, (t, l, st)
                assert st["dense_macs"] == orc.layer_macs(specs[l]) * n
                if specs[0].dtype != "f32" or l == 0:
                    assert st["nnz_elems"] == one.nnz[l], (t, l, st, one.nnz[l])
                    assert st["active_macs"] == one.macs[l], (t, l, st, one.macs[l])
                assert 0 < st["active_out_pixels"] <= st["out_pixels"] and st["nnz_elems"] <= st["in_elems"]
        if check_frames is None or t in check_frames:
            _compare(specs, net, video[t], t)
            # the caller-owned output equals the last tensor
            last = net.tensor(len(specs))
            assert torch.equal(out, last)
    net.close()


# ------------------------------------------------------------------ config 1
def test_cfg1_single_conv_fp32_all_frames():
    specs = wl.single_conv_f32()
    video = wl.block_redraw_sequence()
    _run(specs, video, stats=True)


def _spec(dtype, c_in, hw, c_out, k, s, p, rng, **kw):
    sp = LayerSpec("conv", dtype, c_in, hw[0], hw[1], c_out, k, k, s, p, src=0, **kw)
    if dtype == "f32":
        sp.weight = rng.standard_normal((c_out, c_in, k, k)).astype(np.float32) * np.float32(0.1)
        sp.bias = rng.standard_normal(c_out).astype(np.float32)
    elif dtype == "i8":
        sp.weight = rng.integers(-127, 128, size=(c_out, c_in, k, k)).astype(np.int8)
        sp.bias = rng.integers(-500, 501, size=c_out).astype(np.int32)
    else:
        sp.weight = (rng.integers(0, 2, size=(c_out, c_in, k, k)) * 2 - 1).astype(np.int8)
        sp.bias = rng.integers(-5, 6, size=c_out).astype(np.int32)
    return sp


def _video(dtype, c, hw, frames, n, rng):
    kind = {"f32": "f32_relu", "i8": "i8", "bin": "pm1"}[dtype]
    h, w = hw
    seq = wl.block_redraw_sequence(frames=frames, c=c, hw=max(h, w), frac=0.08, block=3, dtype=kind,
                                   seed=int(rng.integers(1, 1 << 30)), n=n)[:, :, :, :h, :w].copy()
    seq[2] = seq[1]                                  # zero delta
    if dtype == "bin":
        seq[3] = -seq[2]                             # every element changes
    elif dtype == "i8":
        seq[3] = 127 - seq[2]
    else:
        seq[3] = seq[2] + np.float32(0.5)
    return seq


@pytest.mark.parametrize("dtype", ["f32", "i8", "bin"])
@pytest.mark.parametrize("c_in,c_out,hw,k,s,p", [
    (3, 5, (9, 11), 3, 1, 1), (16, 70, (13, 13), 3, 1, 1), (8, 12, (17, 15), 5, 2, 2), (5, 9, (12, 12), 1, 1, 0),
    (4, 8, (20, 19), 1, 2, 0), (3, 6, (35, 35), 11, 4, 0), (3, 8, (30, 30), 7, 2, 3), (40, 33, (7, 7), 3, 1, 0),
    (64, 16, (10, 10), 3, 1, 1)])
def test_single_layer_shapes(dtype, c_in, c_out, hw, k, s, p):
    rng = np.random.default_rng(c_in * 1000 + c_out * 10 + k)
    sp = _spec(dtype, c_in, hw, c_out, k, s, p, rng)
    video = _video(dtype, c_in, hw, 5, 2, rng)
    _run([sp], video, n=2, stats=True)


@pytest.mark.parametrize("dtype", ["i8", "bin"])
@pytest.mark.parametrize("c_in,c_out,hw,k,s,p", [(16, 70, (13, 13), 3, 1, 1), (8, 12, (17, 15), 5, 2, 2), (64, 16, (10, 10), 3, 1, 1),
                                                 (3, 6, (35, 35), 11, 4, 0)])
def test_single_layer_cuda_core_variant(dtype, c_in, c_out, hw, k, s, p):
    """The CUDA-core (dp4a / popcount) variant on layers that would otherwise take the tensor-core one."""
    rng = np.random.default_rng(c_in * 1000 + c_out * 10 + k + 1)
    sp = _spec(dtype, c_in, hw, c_out, k, s, p, rng)
    video = _video(dtype, c_in, hw, 5, 2, rng)
    _run([sp], video, n=2, stats=True, variant="gather")


@pytest.mark.parametrize("dtype,act,pool,shift", [
    ("f32", "relu", (3, 2, 0), -1), ("f32", "relu", (3, 2, 1), -1), ("f32", "none", (2, 2, 0), -1),
    ("f32", "leaky", None, -1), ("f32", "leaky", (2, 2, 0), -1),
    ("i8", "relu", (3, 2, 0), 9), ("i8", "none", None, 10), ("i8", "sign", (3, 2, 0), -1), ("i8", "none", (3, 2, 1), -1),
    ("bin", "sign", None, -1), ("bin", "sign", (3, 2, 0), -1), ("bin", "none", (3, 2, 0), -1)])
def test_single_layer_nonlinearities(dtype, act, pool, shift):
    rng = np.random.default_rng(77)
    sp = _spec(dtype, 12, (15, 14), 40, 3, 1, 1, rng, act=act, pool=pool, shift=shift, theta=3)
    video = _video(dtype, 12, (15, 14), 5, 1, rng)
    _run([sp], video, n=1, stats=True)


def test_keyframe_resets_state_and_dense_path_is_stateless():
    rrm = _rrm()
    specs = wl.single_conv_f32(c_in=8, c_out=8, hw=20)
    video = wl.block_redraw_sequence(frames=6, c=8, hw=20, seed=3)
    _run(specs, video, keyframe_at=(0, 3))
    net = rrm.net_from_specs(specs)
    out, outd = net.new_output(), net.new_output()
    net.step(dev(video[0]), out)
    net.dense(dev(video[4]), outd)
    ref = orc.dense_forward(specs, video[4])[0][1]
    assert np.abs(outd.cpu().numpy() - ref).max() <= F32_TOL * np.abs(ref).max()
    net.step(dev(video[1]), out)
    ref = orc.dense_forward(specs, video[1])[0][1]
    assert np.abs(out.cpu().numpy() - ref).max() <= F32_TOL * np.abs(ref).max()
    net.close()


# ------------------------------------------------------------------ small stacks, every frame, with stats
@pytest.mark.parametrize("name", ["alex_f32", "alex_i8", "resnet_i8", "xnor"])
def test_small_stacks_every_frame(name):
    if name == "alex_f32":
        specs, dt, hw = wl.alexnet_convs("f32", hw=99, scale=8), "f32", 99
    elif name == "alex_i8":
        specs, dt, hw = wl.alexnet_convs("i8", hw=99, scale=8), "i8", 99
    elif name == "resnet_i8":
        specs, dt, hw = wl.resnet18_convs(hw=96, scale=8), "i8", 96
    else:
        specs, dt, hw = wl.xnor_alexnet_convs(hw=99, scale=8), "i8", 99
    n = 2 if name == "resnet_i8" else 1
    video = wl.moving_rect_video(frames=6, hw=hw, dtype=dt, seed=9, n=n, side=(12, 24),
                                 bg_redraw=0.02 if name == "resnet_i8" else 0.0)
    _run(specs, video, n=n, stats=True, keyframe_at=(4,))


# ------------------------------------------------------------------ whole networks: FC layers inside a stack, VGG-16 shape
@pytest.mark.parametrize("name", ["alexnet_full_i8", "alexnet_full_f32", "vgg16_i8", "vgg16_f32"])
def test_second_workloads_every_frame(name):
    dt = "i8" if name.endswith("i8") else "f32"
    if name.startswith("alexnet_full"):
        specs, hw = wl.alexnet_full(dt, hw=99, scale=8, classes=80), 99
    else:
        specs, hw = wl.vgg16_convs(dt, hw=64, scale=8), 64
    video = wl.moving_rect_video(frames=5, hw=hw, dtype=dt, seed=12, side=(10, 20))
    _run(specs, video, stats=True, keyframe_at=(3,))


def test_large_stack_goes_dense_while_nearly_every_pixel_changes():
    """Background noise makes every projection pixel change: after the first measured delta frame the frames
    are evaluated densely (same results), with a delta frame every 16th frame to measure again."""
    rrm = _rrm()
    specs = wl.alexnet_convs("i8")
    video = wl.moving_rect_video(frames=20, hw=227, dtype="i8", seed=33, n=2, bg_redraw=0.10)
    net = rrm.net_from_specs(specs, n=2)
    out = net.new_output()
    variants, counted = [], []
    for t in range(20):
        net.step(dev(video[t]), out)
        st = net.stats(1)                     # synchronises, so the next call sees this frame's counters
        variants.append(st["variant"])
        counted.append(st["nnz_elems"] != -1)
        if t in (0, 1, 2, 16, 19):
            _compare(specs, net, video[t], t)
    assert variants[0] == 2 and counted[0]                # the first frame (every pixel new) is a measured delta frame
    assert all(v == 3 for v in variants[1:16]) and not any(counted[1:16])   # the whole stack dense while the measured activity is high
    # one delta frame measures again (the per-layer choice is off by default: its layers run the sparse product)
    assert variants[16] == 2 and counted[16]
    assert variants[17] == 3 and not counted[17]
    net.close()


@pytest.mark.parametrize("name", ["alex_i8", "resnet_i8", "alex_f32", "xnor"])
def test_layers_choose_between_sparse_and_dense_evaluation_from_their_measured_activity(name):
    """Per-layer choice (variant AUTO): with the thresholds lowered, the layers whose share of projection pixels to
    update is high run a dense evaluation inside the delta step while the others run the sparse product.  Outputs,
    stored projections and counters stay those of Algorithm 1 at every frame, whatever the mix."""
    rrm = _rrm()
    if name == "alex_i8":
        specs, dt, hw, n = wl.alexnet_convs("i8", hw=99, scale=8), "i8", 99, 1
    elif name == "resnet_i8":
        specs, dt, hw, n = wl.resnet18_convs(hw=96, scale=8), "i8", 96, 2
    elif name == "alex_f32":
        specs, dt, hw, n = wl.alexnet_convs("f32", hw=99, scale=8), "f32", 99, 1
    else:
        specs, dt, hw, n = wl.xnor_alexnet_convs(hw=99, scale=8), "i8", 99, 1
    video = wl.moving_rect_video(frames=9, hw=hw, dtype=dt, seed=23, n=n, side=(12, 24))
    net = rrm.net_from_specs(specs, n=n)
    rec = orc.Recurrence(specs, n=n)
    rec.step(np.full_like(video[0], 0))
    out = net.new_output()
    mixes = set()
    for t in range(video.shape[0]):
        net.step(dev(video[t]), out)
        rec.step(video[t])
        vs, acts = [], []
        for l in range(len(specs)):
            st = net.stats(l)                 # synchronises: the next step's choice sees this frame's counters
            vs.append(st["variant"])
            acts.append(st["active_out_pixels"] / st["out_pixels"])
            assert st["error_word"] == 0
            if dt != "f32" or l == 0:
                assert st["nnz_elems"] == rec.nnz[l] and st["active_macs"] == rec.macs[l], (t, l, st, rec.nnz[l], rec.macs[l])
        mixes.add(tuple(v == 3 for v in vs))
        _compare(specs, net, video[t], t)
        if t == 2:
            # thresholds between this video's measured per-layer activities, so that the layers really split
            a = sorted(set(acts))
            assert len(a) >= 2, acts
            thr = 0.5 * (a[len(a) // 2 - 1] + a[len(a) // 2])
            net.set_options(layer_dense_activity=thr, layer_delta_activity=0.95 * thr)
    assert any(any(m) and not all(m) for m in mixes), mixes       # some frame ran a real mix of the two evaluations
    # ... and a chunk of frames with the mix chosen at its start
    more = wl.moving_rect_video(frames=13, hw=hw, dtype=dt, seed=23, n=n, side=(12, 24))
    outs = net.new_output(frames=4)
    net.step_seq(dev(np.ascontiguousarray(more[9:13])), outs, 4)
    _compare(specs, net, more[12], 12)
    net.close()


# ------------------------------------------------------------------ full-size configs, sampled frames
def test_cfg3_alexnet_fp32_full_size():
    specs = wl.alexnet_convs("f32")
    video = wl.moving_rect_video(frames=64, hw=227, dtype="f32", seed=31)
    _run(specs, video, check_frames={0, 1, 2, 17, 63})


def test_cfg3_alexnet_int8_full_size():
    specs = wl.alexnet_convs("i8")
    video = wl.moving_rect_video(frames=64, hw=227, dtype="i8", seed=32)
    _run(specs, video, check_frames={0, 1, 30, 63}, stats_frames={30})


def test_cfg3_alexnet_int8_early_layers_sparse_late_layers_dense():
    """On the moving-rectangle video the first layers update a fifth to a half of their projection pixels, the last
    ones nearly all: with the thresholds at 0.75 / 0.60 the library settles on the sparse product for conv1-2 and a
    dense evaluation for conv5, inside the same delta step."""
    rrm = _rrm()
    specs = wl.alexnet_convs("i8")
    video = wl.moving_rect_video(frames=20, hw=227, dtype="i8", seed=32)
    net = rrm.net_from_specs(specs)
    net.set_options(layer_dense_activity=0.75, layer_delta_activity=0.60)
    out = net.new_output()
    # (frame 0 changes every pixel, so this stack of > 1 GMAC is evaluated densely as a whole for the next 15 frames;
    # frame 16 measures again, and from frame 17 on every layer follows its own activity)
    for t in range(20):
        net.step(dev(video[t]), out)
        vs = [net.stats(l)["variant"] for l in range(len(specs))]
    assert vs[0] == 2 and vs[1] == 2 and vs[4] == 3, vs
    act = [net.stats(l)["active_out_pixels"] / net.stats(l)["out_pixels"] for l in range(len(specs))]
    assert act[0] < 0.6 and act[4] > 0.75, act
    _compare(specs, net, video[19], 19)
    net.close()


def test_cfg4_resnet18_int8_batch4():
    specs = wl.resnet18_convs()
    video = wl.moving_rect_video(frames=64, hw=224, dtype="i8", seed=41, n=4, bg_redraw=0.02)
    _run(specs, video, n=4, check_frames={0, 1, 63})


def test_cfg4_resnet18_int8_batch4_every_frame_through_the_delta_kernels():
    """The same stack with the delta / dense switch off (variant "tensor"): every frame goes through the sparse
    product at partial density, every layer's projection is compared at five frames, the counters at two."""
    specs = wl.resnet18_convs()
    video = wl.moving_rect_video(frames=64, hw=224, dtype="i8", seed=41, n=4, bg_redraw=0.02)
    _run(specs, video, n=4, check_frames={0, 1, 16, 32, 63}, stats_frames={16, 63}, variant="tensor")


def test_cfg5_xnor_alexnet_128_frames():
    specs = wl.xnor_alexnet_convs()
    video = wl.moving_rect_video(frames=128, hw=227, dtype="i8", seed=51)
    _run(specs, video, check_frames={0, 1, 64, 127}, stats_frames={64})


# ------------------------------------------------------------------ chunks of frames through a stack (frames overlap layer by layer)
@pytest.mark.parametrize("by_layer", [False, True])
@pytest.mark.parametrize("name", ["alex_f32", "alex_i8", "resnet_i8", "xnor", "alexnet_full_i8"])
def test_stack_chunks_of_frames_equal_frame_by_frame(name, by_layer, monkeypatch):
    """rrm_net_step_seq on a stack runs the frames of a chunk as one graph in which consecutive frames overlap, or
    (by_layer: forced here, chosen by the library for long chunks of few streams) every layer over all frames of the
    chunk in one launch; every frame's output, the state after each chunk and the last frame's counters are those of
    Algorithm 1."""
    if by_layer:
        monkeypatch.setenv("RRM_CHUNK_BY_LAYER", "1")
    rrm = _rrm()
    if name == "alex_f32":
        specs, dt, hw = wl.alexnet_convs("f32", hw=99, scale=8), "f32", 99
    elif name == "alex_i8":
        specs, dt, hw = wl.alexnet_convs("i8", hw=99, scale=8), "i8", 99
    elif name == "resnet_i8":
        specs, dt, hw = wl.resnet18_convs(hw=96, scale=8), "i8", 96
    elif name == "xnor":
        specs, dt, hw = wl.xnor_alexnet_convs(hw=99, scale=8), "i8", 99
    else:
        specs, dt, hw = wl.alexnet_full("i8", hw=99, scale=8, classes=80), "i8", 99
    n = 2 if name == "resnet_i8" else 1
    video = wl.moving_rect_video(frames=17, hw=hw, dtype=dt, seed=19, n=n, side=(12, 24),
                                 bg_redraw=0.02 if name == "resnet_i8" else 0.0)
    net = rrm.net_from_specs(specs, n=n)
    rec = orc.Recurrence(specs, n=n)
    rec.step(np.full_like(video[0], 0))
    frames = dev(np.ascontiguousarray(video))
    t0 = 0
    for T in (5, 5, 2, 4):                    # the same length twice (graph reuse), then other lengths
        outs = net.new_output(frames=T)
        net.step_seq(frames[t0:t0 + T], outs, T)
        for i in range(T):
            rec.step(video[t0 + i])
            want = orc.dense_forward(specs, video[t0 + i])[0][len(specs)]
            got = outs[i].cpu().numpy()
            if dt == "f32":
                assert float(np.abs(got - want).max()) <= F32_TOL * max(1e-30, float(np.abs(want).max())), (t0 + i)
            elif _out_kind(specs[-1]) == "bin":
                np.testing.assert_array_equal(unpack_bits_nhwc(got.view(np.uint32), specs[-1].c_out), want, err_msg=f"frame {t0 + i}")
            else:
                np.testing.assert_array_equal(got.astype(np.int64), want, err_msg=f"frame {t0 + i}")
        t0 += T
        _compare(specs, net, video[t0 - 1], t0 - 1)          # every layer's stored projection and tensor after the chunk
        for l in range(len(specs)):
            st = net.stats(l)
            assert st["error_word"] == 0
            if dt != "f32" or l == 0:
                assert st["nnz_elems"] == rec.nnz[l] and st["active_macs"] == rec.macs[l], (t0, l, st)
    # frame-by-frame stepping carries on from the chunk's state
    out = net.new_output()
    net.step(dev(video[16]), out)
    _compare(specs, net, video[16], 16)
    # dense chunks leave the state alone
    outs = net.new_output(frames=3)
    net.dense_seq(frames[2:5], outs, 3)
    for i in range(3):
        want = orc.dense_forward(specs, video[2 + i])[0][len(specs)]
        got = outs[i].cpu().numpy()
        if dt == "f32":
            assert float(np.abs(got - want).max()) <= F32_TOL * max(1e-30, float(np.abs(want).max()))
        elif _out_kind(specs[-1]) == "bin":
            np.testing.assert_array_equal(unpack_bits_nhwc(got.view(np.uint32), specs[-1].c_out), want)
        else:
            np.testing.assert_array_equal(got.astype(np.int64), want)
    _compare(specs, net, video[16], 16)
    net.close()


@pytest.mark.parametrize("name", ["cfg1", "cfg3_f32", "cfg3_i8", "cfg5", "cfg4"])
def test_full_size_stacks_in_chunks_of_32_frames(name):
    """The full-size configurations in the launch configuration the bench times for chunks: 32 frames per
    rrm_net_step_seq call.  First chunk and second chunk on the delta path (thresholds out of reach), the third as the
    library chooses; sampled frames' outputs against the dense definition, every layer's state after each chunk, and
    the last frame's counters of the second chunk against Algorithm 1 brought to the frame before by a dense pass."""
    rrm = _rrm()
    n = 1
    if name == "cfg1":
        specs, dt, hw = wl.single_conv_f32(), "f32", 56
    elif name == "cfg3_f32":
        specs, dt, hw = wl.alexnet_convs("f32"), "f32", 227
    elif name == "cfg3_i8":
        specs, dt, hw = wl.alexnet_convs("i8"), "i8", 227
    elif name == "cfg5":
        specs, dt, hw = wl.xnor_alexnet_convs(), "i8", 227
    else:
        specs, dt, hw, n = wl.resnet18_convs(), "i8", 224, 4
    if name == "cfg1":
        video = wl.block_redraw_sequence(frames=96, seed=61)
    else:
        video = wl.moving_rect_video(frames=96, hw=hw, dtype=dt, seed=61, n=n, bg_redraw=0.02 if name == "cfg4" else 0.0)
    net = rrm.net_from_specs(specs, n=n)
    defaults = net.options()
    net.set_options(chunk_dense_activity=2.0, stack_dense_activity=2.0)
    frames = dev(np.ascontiguousarray(video))
    outs = net.new_output(frames=32)
    for k in range(3):
        if k == 2:
            net.set_options(chunk_dense_activity=defaults["chunk_dense_activity"], stack_dense_activity=defaults["stack_dense_activity"])
        net.step_seq(frames[32 * k:32 * k + 32], outs, 32)
        sts = [net.stats(l) for l in range(len(specs))]
        assert all(st["error_word"] == 0 for st in sts)
        for i in ((0, 13, 31) if k < 2 else (0, 31)):
            want = orc.dense_forward(specs, video[32 * k + i])[0][len(specs)]
            got = outs[i].cpu().numpy()
            if dt == "f32":
                assert float(np.abs(got - want).max()) <= F32_TOL * max(1e-30, float(np.abs(want).max())), (k, i)
            elif _out_kind(specs[-1]) == "bin":
                np.testing.assert_array_equal(unpack_bits_nhwc(got.view(np.uint32), specs[-1].c_out), want, err_msg=f"chunk {k} frame {i}")
            else:
                np.testing.assert_array_equal(got.astype(np.int64), want, err_msg=f"chunk {k} frame {i}")
        _compare(specs, net, video[32 * k + 31], 32 * k + 31)
        if k == 1:
            one = orc.Recurrence(specs, n=n)
            one.reset_to(video[62])
            one.step(video[63])
            for l, st in enumerate(sts):
                assert st["variant"] != 3 and st["nnz_elems"] != -1, (l, st)
                if dt != "f32" or l == 0:
                    assert st["nnz_elems"] == one.nnz[l] and st["active_macs"] == one.macs[l], (l, st, one.nnz[l], one.macs[l])
    net.close()


def test_large_stack_chunks_go_dense_while_nearly_every_pixel_changes():
    """The density switch of a large stack, chunk by chunk: the chunk after a measured high-activity delta chunk is
    evaluated densely (a sequence of precise inferences that replace the state); outputs and state stay exact."""
    rrm = _rrm()
    specs = wl.alexnet_convs("i8")
    video = wl.moving_rect_video(frames=13, hw=227, dtype="i8", seed=34, n=2, bg_redraw=0.10)
    net = rrm.net_from_specs(specs, n=2)
    frames = dev(np.ascontiguousarray(video))
    variants = []
    for k in range(3):
        outs = net.new_output(frames=4)
        net.step_seq(frames[4 * k:4 * k + 4], outs, 4)
        st = net.stats(1)                     # synchronises, so the next call sees this chunk's counters
        variants.append(st["variant"])
        assert (st["nnz_elems"] == -1) == (st["variant"] == 3)
        for i in (0, 3):
            want = orc.dense_forward(specs, video[4 * k + i])[0][len(specs)]
            np.testing.assert_array_equal(outs[i].cpu().numpy().astype(np.int64), want, err_msg=f"frame {4 * k + i}")
        _compare(specs, net, video[4 * k + 3], 4 * k + 3)
    assert variants[0] == 2 and variants[1] == 3 and variants[2] == 3, variants
    out = net.new_output()
    net.step(dev(video[12]), out)             # frame by frame from the state the dense chunks left
    _compare(specs, net, video[12], 12)
    net.close()


def test_long_chunks_of_a_tensor_core_stack_go_dense_from_the_measured_activity():
    """rrm_options.chunk_dense_activity: after a delta chunk that measured a high share of pixels to update, the next
    long chunks of an int8 stack are evaluated densely, batched over their frames; outputs and state stay exact, and
    with the threshold out of reach the library stays on the delta path."""
    rrm = _rrm()
    specs = wl.alexnet_convs("i8", hw=99, scale=8)
    video = wl.moving_rect_video(frames=65, hw=99, dtype="i8", seed=43, n=1, side=(12, 24), bg_redraw=0.10)
    net = rrm.net_from_specs(specs, n=1)
    assert abs(net.options()["chunk_dense_activity"] - 0.40) < 1e-6
    frames = dev(np.ascontiguousarray(video))
    variants = []
    for k in range(4):
        if k == 3:
            net.set_options(chunk_dense_activity=2.0)
        outs = net.new_output(frames=16)
        net.step_seq(frames[16 * k:16 * k + 16], outs, 16)
        st = net.stats(1)                     # synchronises, so the next call sees this chunk's counters
        variants.append(st["variant"])
        for i in (0, 7, 15):
            want = orc.dense_forward(specs, video[16 * k + i])[0][len(specs)]
            np.testing.assert_array_equal(outs[i].cpu().numpy().astype(np.int64), want, err_msg=f"frame {16 * k + i}")
        _compare(specs, net, video[16 * k + 15], 16 * k + 15)
    assert variants[0] != 3 and variants[1] == 3 and variants[2] == 3 and variants[3] != 3, variants
    out = net.new_output()
    net.step(dev(video[64]), out)
    _compare(specs, net, video[64], 64)
    net.close()


def test_dense_chunks_longer_than_one_batch():
    """Dense chunks are batched over their frames, 32 at most per launch: a chunk of 40 frames of two streams goes in
    two parts.  rrm_net_dense_seq leaves the state alone; a chunk that the density switch evaluates densely leaves
    the state at its last frame."""
    rrm = _rrm()
    specs = wl.alexnet_convs("i8", hw=67, scale=8)
    video = wl.moving_rect_video(frames=81, hw=67, dtype="i8", seed=47, n=2, side=(8, 16))
    net = rrm.net_from_specs(specs, n=2)
    frames = dev(np.ascontiguousarray(video))
    out = net.new_output()
    net.keyframe(frames[0], out)
    outs = net.new_output(frames=40)
    net.dense_seq(frames[1:41], outs, 40)
    for i in (0, 19, 20, 39):
        want = orc.dense_forward(specs, video[1 + i])[0][len(specs)]
        np.testing.assert_array_equal(outs[i].cpu().numpy().astype(np.int64), want, err_msg=f"frame {1 + i}")
    _compare(specs, net, video[0], 0)                       # the state is still the keyframe's
    net.set_options(chunk_dense_activity=0.0)               # every measured activity sends the next chunk to the dense evaluation
    net.step_seq(frames[1:41], outs, 40)                    # (nothing measured yet: the delta path)
    assert net.stats(1)["variant"] != 3
    _compare(specs, net, video[40], 40)
    net.step_seq(frames[41:81], outs, 40)
    assert net.stats(1)["variant"] == 3
    for i in (0, 21, 39):
        want = orc.dense_forward(specs, video[41 + i])[0][len(specs)]
        np.testing.assert_array_equal(outs[i].cpu().numpy().astype(np.int64), want, err_msg=f"frame {41 + i}")
    _compare(specs, net, video[80], 80)
    net.close()


def test_stack_chunks_through_the_pipelined_host_entry_point():
    """Host buffers in, host buffers out, calls queued without waiting: a stack's chunks through
    rrm_net_step_seq_host_async deliver every frame's output."""
    rrm = _rrm()
    specs = wl.alexnet_convs("i8", hw=99, scale=8)
    video = wl.moving_rect_video(frames=12, hw=99, dtype="i8", seed=23, n=1, side=(12, 24))
    net = rrm.net_from_specs(specs, n=1)
    ins = [torch.from_numpy(np.ascontiguousarray(video[a:a + 4])).pin_memory() for a in (0, 4, 8)]
    shape = tuple(net.new_output(frames=4).shape)
    outs = [torch.empty(shape, dtype=torch.int8).pin_memory() for _ in range(3)]
    for x, y in zip(ins, outs):
        net.step_seq_host_async(x, y, 4)
    net.host_sync()
    for k, y in enumerate(outs):
        for i in range(4):
            want = orc.dense_forward(specs, video[4 * k + i])[0][len(specs)]
            np.testing.assert_array_equal(y[i].numpy().astype(np.int64), want, err_msg=f"frame {4 * k + i}")
    net.close()


def test_stack_chunk_longer_than_the_arenas_held():
    """More frames in one call than there are per-frame arenas: arenas are reused, each cleared by the frame that
    takes it over; outputs and state are unchanged."""
    rrm = _rrm()
    specs = wl.alexnet_convs("i8", hw=67, scale=8)
    video = wl.moving_rect_video(frames=71, hw=67, dtype="i8", seed=29, n=1, side=(8, 16))
    net = rrm.net_from_specs(specs, n=1)
    rec = orc.Recurrence(specs, n=1)
    rec.step(np.full_like(video[0], 0))
    frames = dev(np.ascontiguousarray(video))
    outs = net.new_output(frames=70)
    net.step_seq(frames[:70], outs, 70)
    for t in range(70):
        rec.step(video[t])
        if t in (0, 1, 33, 64, 65, 69):
            want = orc.dense_forward(specs, video[t])[0][len(specs)]
            np.testing.assert_array_equal(outs[t].cpu().numpy().astype(np.int64), want, err_msg=f"frame {t}")
    _compare(specs, net, video[69], 69)
    for l in range(len(specs)):
        st = net.stats(l)
        assert st["error_word"] == 0 and st["nnz_elems"] == rec.nnz[l] and st["active_macs"] == rec.macs[l], (l, st)
    out = net.new_output()
    net.step(dev(video[70]), out)
    _compare(specs, net, video[70], 70)
    net.close()


# ------------------------------------------------------------------ explicit batch normalisation as part of f (Sec. 4.5)
@pytest.mark.parametrize("name", ["alex_f32", "resnet_i8", "vgg_i8"])
def test_explicit_bn_stacks_every_frame(name):
    """Stacks whose layers keep their batch normalisation explicit (per-channel affine before requantisation /
    activation / pooling): projections, tensors and counters against the oracle at every frame, a keyframe in between."""
    if name == "alex_f32":
        specs, dt, hw, n = wl.alexnet_convs("f32", hw=99, scale=8), "f32", 99, 1
    elif name == "resnet_i8":
        specs, dt, hw, n = wl.resnet18_convs(hw=96, scale=8), "i8", 96, 2
    else:
        specs, dt, hw, n = wl.vgg16_convs("i8", hw=64, scale=8), "i8", 64, 1
    wl.with_explicit_bn(specs)
    assert all(s.bn_scale is not None for s in specs)
    video = wl.moving_rect_video(frames=6, hw=hw, dtype=dt, seed=29, n=n, side=(10, 20))
    _run(specs, video, n=n, stats=True, keyframe_at=(3,))


@pytest.mark.parametrize("by_layer", [False, True])
@pytest.mark.parametrize("name", ["alex_f32", "resnet_i8"])
def test_explicit_bn_stacks_in_chunks(name, by_layer, monkeypatch):
    """The same stacks through rrm_net_step_seq, frame-pipelined and layer by layer over all frames of a chunk:
    every frame's output, then projections and tensors after the chunk."""
    if by_layer:
        monkeypatch.setenv("RRM_CHUNK_BY_LAYER", "1")
    rrm = _rrm()
    if name == "alex_f32":
        specs, dt, hw, n = wl.alexnet_convs("f32", hw=99, scale=8), "f32", 99, 1
    else:
        specs, dt, hw, n = wl.resnet18_convs(hw=96, scale=8), "i8", 96, 2
    wl.with_explicit_bn(specs)
    video = wl.moving_rect_video(frames=9, hw=hw, dtype=dt, seed=37, n=n, side=(10, 20))
    net = rrm.net_from_specs(specs, n=n)
    frames = dev(np.ascontiguousarray(video))
    t0 = 0
    for T in (5, 4):
        outs = net.new_output(frames=T)
        net.step_seq(frames[t0:t0 + T], outs, T)
        for i in range(T):
            want = orc.dense_forward(specs, video[t0 + i])[0][len(specs)]
            got = outs[i].cpu().numpy()
            if dt == "f32":
                assert float(np.abs(got - want).max()) <= F32_TOL * max(1e-30, float(np.abs(want).max())), t0 + i
            else:
                np.testing.assert_array_equal(got.astype(np.int64), want, err_msg=f"frame {t0 + i}")
        t0 += T
        _compare(specs, net, video[t0 - 1], t0 - 1)
    for l in range(len(specs)):
        assert net.stats(l)["error_word"] == 0
    net.close()


def test_explicit_bn_equals_the_folded_stack_on_the_gpu():
    """fp32: the stack with its affines unfolded and the stack with them folded into filters and bias give the same
    tensors within the fp32 tolerance, on the library's delta path."""
    rrm = _rrm()
    specs = wl.with_explicit_bn(wl.alexnet_convs("f32", hw=99, scale=8))
    folded = wl.fold_bn_f32(specs)
    video = wl.moving_rect_video(frames=5, hw=99, dtype="f32", seed=30, side=(10, 20))
    a, b = rrm.net_from_specs(specs), rrm.net_from_specs(folded)
    oa, ob = a.new_output(), b.new_output()
    for t in range(5):
        a.step(dev(video[t]), oa)
        b.step(dev(video[t]), ob)
        scale = float(ob.abs().max())
        assert float((oa - ob).abs().max()) <= 5 * F32_TOL * max(scale, 1e-6), t
    # removing the affine again gives the plain stack's fresh state
    plain = wl.alexnet_convs("f32", hw=99, scale=8)
    for l in range(len(specs)):
        a.set_affine(l, None, None)
    a.step(dev(video[0]), oa)
    want = orc.dense_forward(plain, video[0])[0][len(plain)]
    assert float(np.abs(oa.cpu().numpy() - want).max()) <= F32_TOL * float(np.abs(want).max())
    a.close(); b.close()


def test_affine_is_rejected_where_it_is_not_defined():
    rrm = _rrm()
    specs = wl.xnor_alexnet_convs(hw=99, scale=8)
    net = rrm.net_from_specs(specs)
    z = torch.zeros(specs[0].c_out, dtype=torch.int32, device="cuda")
    with pytest.raises(rrm.RRMError):
        net.set_affine(0, z, z)               # a sign layer
    with pytest.raises(rrm.RRMError):
        net.set_affine(0, z, None)
    net.close()


# ------------------------------------------------------------------ fp32 results are reproducible bit for bit
@pytest.mark.parametrize("name", ["cfg1", "alex_f32"])
def test_fp32_projections_are_bitwise_reproducible(name):
    """Layers whose K range is split over CTAs add their shares' partial sums in a fixed order, so two runs over the
    same frames leave bit-identical projections (the race detector of last resort: any unordered float addition or
    data race would show here)."""
    rrm = _rrm()
    if name == "cfg1":
        specs, video = wl.single_conv_f32(), wl.block_redraw_sequence()
    else:
        specs, video = wl.alexnet_convs("f32", hw=131, scale=4), wl.moving_rect_video(frames=6, hw=131, dtype="f32", seed=3, side=(12, 24))
    runs = []
    for rep in range(3):
        net = rrm.net_from_specs(specs, variant="tensor")      # (no density switch: every frame through the delta kernels)
        out = net.new_output()
        for t in range(video.shape[0]):
            net.step(dev(video[t]), out)
        runs.append([net.projection(l).clone() for l in range(len(specs))] + [out.clone()])
        net.close()
    for other in runs[1:]:
        for a, b in zip(runs[0], other):
            assert torch.equal(a, b)


# ------------------------------------------------------------------ chunk forms: layer by layer, frame-pipelined, in place
def _two_layer_stack(dtype, rng):
    """Layer 0 reads a multi-channel input of the given type (the import kernels of every input layout) and pools with
    a window that leaves trailing projection rows outside every window; layer 1 reads its output."""
    if dtype == "bin":
        a = _spec("bin", 40, (15, 14), 36, 3, 1, 1, rng, act="sign", pool=(3, 2, 0), theta=2)
        b = _spec("bin", 36, (7, 6), 20, 3, 1, 1, rng, act="sign", theta=1)
    elif dtype == "i8":
        a = _spec("i8", 16, (16, 14), 40, 3, 1, 1, rng, act="relu", pool=(3, 2, 0), shift=11)
        b = _spec("i8", 40, (7, 6), 24, 3, 1, 1, rng, act="none")
    else:
        a = _spec("f32", 12, (16, 14), 40, 3, 1, 1, rng, act="relu", pool=(2, 2, 0))
        b = _spec("f32", 40, (8, 7), 24, 3, 1, 1, rng, act="leaky")
    b.src = 1
    return [a, b]


@pytest.mark.parametrize("form", ["layer_by_layer", "pipelined", "in_place"])
@pytest.mark.parametrize("dtype", ["f32", "i8", "bin"])
def test_chunk_forms_agree_with_the_oracle(dtype, form, monkeypatch):
    """rrm_net_step_seq on a delta chunk has three forms (every kernel over all frames of the chunk; frames
    overlapping in one graph with the frame's product kept apart; the same adding in place).  Each must give every
    frame's output, the state after the chunk and the last frame's counters of Algorithm 1 - also across a frame
    without change and a frame in which everything changes, for every input layout, two streams."""
    if form == "layer_by_layer":
        monkeypatch.setenv("RRM_CHUNK_BY_LAYER", "1")
    elif form == "pipelined":
        monkeypatch.setenv("RRM_CHUNK_PIPELINED", "1")
    elif form == "in_place":
        monkeypatch.setenv("RRM_CHUNK_INPLACE", "1")
    rrm = _rrm()
    rng = np.random.default_rng({"f32": 5, "i8": 6, "bin": 7}[dtype])
    specs = _two_layer_stack(dtype, rng)
    s0 = specs[0]
    video = _video(dtype, s0.c_in, (s0.h, s0.w), 10, 2, rng)
    net = rrm.net_from_specs(specs, n=2)
    rec = orc.Recurrence(specs, n=2)
    rec.step(np.full_like(video[0], -1 if dtype == "bin" else 0))
    packed = [_frame_to_dev(specs, video[t]) for t in range(video.shape[0])]
    t0 = 0
    for T in (4, 3, 2):
        frames = torch.stack(packed[t0:t0 + T]).contiguous()
        outs = net.new_output(frames=T)
        net.step_seq(frames, outs, T)
        for i in range(T):
            rec.step(video[t0 + i])
            want = orc.dense_forward(specs, video[t0 + i])[0][len(specs)]
            got = outs[i].cpu().numpy()
            if dtype == "f32":
                assert float(np.abs(got - want).max()) <= F32_TOL * max(1e-30, float(np.abs(want).max())), t0 + i
            elif dtype == "bin":
                np.testing.assert_array_equal(unpack_bits_nhwc(got.view(np.uint32), specs[-1].c_out), want, err_msg=f"frame {t0 + i}")
            else:
                np.testing.assert_array_equal(got.astype(np.int64), want, err_msg=f"frame {t0 + i}")
        t0 += T
        _compare(specs, net, video[t0 - 1], t0 - 1)
        for l in range(len(specs)):
            st = net.stats(l)
            assert st["error_word"] == 0
            if dtype != "f32" or l == 0:
                assert st["nnz_elems"] == rec.nnz[l] and st["active_macs"] == rec.macs[l], (form, t0, l, st, rec.nnz[l], rec.macs[l])
    out = net.new_output()
    net.step(packed[9], out)                  # a single step carries on from the chunk's state
    _compare(specs, net, video[9], 9)
    net.close()
