"""GPU parity of the fused delta-FC path against the CPU oracle (bit-exact int32)."""
import numpy as np
import pytest
import torch

import workloads as wl
from workloads.nets import LayerSpec
from oracle import rrm_oracle as orc
from helpers import dev

pytestmark = pytest.mark.gpu


def _rrm():
    import paper_1802_09723_b200 as rrm
    return rrm


def _run_sequence(spec, seq, n, keyframe_first=False):
    rrm = _rrm()
    layer = rrm.layer_from_spec(spec, n=n)
    rec = orc.Recurrence([spec], n=n)
    Y = layer.new_output()
    for t in range(seq.shape[0]):
        x = dev(seq[t])
        if t == 0 and keyframe_first:
            layer.keyframe(x, Y)
        else:
            layer.step(x, Y)
        tens_d, P_d = orc.dense_forward([spec], seq[t])
        got = Y.cpu().numpy().astype(np.int64)
        np.testing.assert_array_equal(got, tens_d[1].astype(np.int64), err_msg=f"frame {t}")
        np.testing.assert_array_equal(layer.projection(0).cpu().numpy().astype(np.int64), P_d[0])
        rec.step(seq[t])
        if not (t == 0 and keyframe_first):
            st = layer.stats(0)
            assert st["nnz_elems"] == rec.nnz[0], (t, st)
            assert st["active_macs"] == rec.macs[0]
            assert st["error_word"] == 0
    layer.close()


@pytest.mark.parametrize("rho", [0.01, 0.05, 0.20])
def test_fc6_int8_all_frames_bit_exact(rho):
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=32, rho=rho, seed=21)
    _run_sequence(spec, seq, 1)


def test_fc6_keyframe_then_steps_and_two_streams():
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=6, rho=0.05, seed=22, n=2)
    _run_sequence(spec, seq, 2, keyframe_first=True)


def test_fc6_many_streams_take_the_two_kernel_form():
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=5, rho=0.05, seed=25, n=5)
    seq[3, 2] = seq[2, 2]                 # one stream with zero delta in one frame
    _run_sequence(spec, seq, 5, keyframe_first=True)


@pytest.mark.parametrize("c_in,c_out,shift,act", [(64, 48, -1, "none"), (160, 528, 6, "relu"),
                                                  (1024 + 32, 16, 5, "none"), (32, 1040, -1, "none")])
def test_fc_small_and_ragged_shapes(c_in, c_out, shift, act):
    rng = np.random.default_rng(c_in + c_out)
    spec = LayerSpec("fc", "i8", c_in, 1, 1, c_out, act=act, shift=shift, src=0)
    spec.weight = rng.integers(-127, 128, size=(c_out, c_in, 1, 1)).astype(np.int8)
    spec.bias = rng.integers(-500, 501, size=c_out).astype(np.int32)
    seq = wl.fc_run_sequence(frames=5, c_in=c_in, rho=0.25, run=8, seed=c_in, n=3)
    seq[3] = seq[2]                       # a frame with zero delta
    seq[4] = 127 - seq[3]                 # every entry changes, deltas up to +-127
    _run_sequence(spec, seq, 3)


def test_fc_full_range_inputs_need_split_deltas():
    """Inputs spanning [-127,127] give deltas up to +-254, beyond one int8 factor."""
    rng = np.random.default_rng(9)
    spec = LayerSpec("fc", "i8", 96, 1, 1, 64, src=0)
    spec.weight = rng.integers(-127, 128, size=(64, 96, 1, 1)).astype(np.int8)
    spec.bias = np.zeros(64, dtype=np.int32)
    a = rng.integers(-127, 128, size=(1, 96)).astype(np.int8)
    seq = np.stack([a, (-a).astype(np.int8), a])
    seq[1, 0, :4] = [127, -127, 127, -127]
    seq[2, 0, :4] = [-127, 127, -127, 127]
    _run_sequence(spec, seq, 1)


def test_fc_dense_path_leaves_state_untouched():
    rrm = _rrm()
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=3, rho=0.05, seed=23)
    layer = rrm.layer_from_spec(spec)
    Y, Yd = layer.new_output(), layer.new_output()
    layer.step(dev(seq[0]), Y)
    layer.dense(dev(seq[2]), Yd)          # unrelated frame through the dense path
    np.testing.assert_array_equal(Yd.cpu().numpy(), orc.dense_forward([spec], seq[2])[0][1])
    layer.step(dev(seq[1]), Y)            # state must still be that of frame 0
    np.testing.assert_array_equal(Y.cpu().numpy(), orc.dense_forward([spec], seq[1])[0][1])
    layer.close()


def test_fc_step_host_matches_device_call():
    rrm = _rrm()
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=3, rho=0.2, seed=24)
    layer = rrm.layer_from_spec(spec)
    out = torch.empty((1, 4096, 1, 1), dtype=torch.int32).pin_memory()
    for t in range(3):
        layer.step_host(torch.from_numpy(seq[t]).pin_memory(), out)
        np.testing.assert_array_equal(out.numpy(), orc.dense_forward([spec], seq[t])[0][1])
    layer.close()


# ------------------------------------------------------------------ chunks of frames in one call
def _run_chunks(spec, seq, n, chunks):
    """Feeds `seq` ([F][n][c_in]) in chunks of the given lengths and checks every frame's output,
    the stored projection after each chunk and the summed counters against the oracle."""
    rrm = _rrm()
    layer = rrm.layer_from_spec(spec, n=n)
    rec = orc.Recurrence([spec], n=n)
    frames = dev(seq)
    t0 = 0
    for T in chunks:
        Y = layer.new_output(frames=T)
        layer.step_seq(frames[t0:t0 + T], Y, T)
        got = Y.cpu().numpy().astype(np.int64)
        nnz = macs = 0
        for i in range(T):
            tens_d, P_d = orc.dense_forward([spec], seq[t0 + i])
            np.testing.assert_array_equal(got[i], tens_d[1].astype(np.int64), err_msg=f"frame {t0 + i}")
            rec.step(seq[t0 + i])
            nnz += rec.nnz[0]
            macs += rec.macs[0]
        np.testing.assert_array_equal(layer.projection(0).cpu().numpy().astype(np.int64), P_d[0])
        st = layer.stats(0)
        assert st["nnz_elems"] == nnz and st["active_macs"] == macs and st["error_word"] == 0, st
        assert st["in_elems"] == T * n * spec.c_in
        t0 += T
    # a single-frame step after the chunks continues from the same state
    if t0 < seq.shape[0]:
        Y1 = layer.new_output()
        layer.step(frames[t0], Y1)
        np.testing.assert_array_equal(Y1.cpu().numpy().astype(np.int64),
                                      orc.dense_forward([spec], seq[t0])[0][1].astype(np.int64))
    layer.close()


@pytest.mark.parametrize("rho", [0.01, 0.05, 0.20])
def test_fc6_chunk_of_32_frames_bit_exact(rho):
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=32, rho=rho, seed=21)
    _run_chunks(spec, seq, 1, [32])


def test_fc6_chunks_of_uneven_length_and_streams():
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=14, rho=0.05, seed=26, n=3)
    seq[5, 1] = seq[4, 1]                 # one stream with zero delta in one frame
    seq[9] = seq[8]                       # a frame with zero delta in every stream
    _run_chunks(spec, seq, 3, [1, 7, 2, 3])


@pytest.mark.parametrize("c_in,c_out,shift,act", [(64, 48, -1, "none"), (160, 528, 6, "relu"),
                                                  (1024 + 32, 16, 5, "none"), (32, 1040, -1, "none"),
                                                  (16384, 128, -1, "none")])
def test_fc_chunks_small_and_ragged_shapes(c_in, c_out, shift, act):
    rng = np.random.default_rng(c_in + c_out + 1)
    spec = LayerSpec("fc", "i8", c_in, 1, 1, c_out, act=act, shift=shift, src=0)
    spec.weight = rng.integers(-127, 128, size=(c_out, c_in, 1, 1)).astype(np.int8)
    spec.bias = rng.integers(-500, 501, size=c_out).astype(np.int32)
    seq = wl.fc_run_sequence(frames=7, c_in=c_in, rho=0.25, run=8, seed=c_in, n=2)
    seq[3] = seq[2]                       # zero delta
    seq[4] = 127 - seq[3]                 # every entry changes
    seq[5] = -seq[4]                      # deltas up to +-254 (split into two int8 factors)
    _run_chunks(spec, seq, 2, [3, 3])


def test_fc_chunk_equals_single_frame_steps_and_dense_chunk_is_stateless():
    rrm = _rrm()
    spec = wl.fc6_i8(c_in=2048, c_out=1024)[0]
    seq = wl.fc_run_sequence(frames=9, c_in=2048, rho=0.1, seed=27, n=2)
    a, b = rrm.layer_from_spec(spec, n=2), rrm.layer_from_spec(spec, n=2)
    frames = dev(seq)
    Ya, Yb = a.new_output(frames=8), b.new_output()
    a.step_seq(frames[:8], Ya, 8)
    for t in range(8):
        b.step(frames[t], Yb)
        assert torch.equal(Ya[t], Yb), t
    assert torch.equal(a.projection(0), b.projection(0))
    # dense chunk: every frame on its own, state untouched
    Yd = a.new_output(frames=3)
    a.dense_seq(frames[2:5], Yd, 3)
    for i in range(3):
        np.testing.assert_array_equal(Yd[i].cpu().numpy(), orc.dense_forward([spec], seq[2 + i])[0][1])
    Y1 = a.new_output()
    a.step(frames[8], Y1)
    np.testing.assert_array_equal(Y1.cpu().numpy(), orc.dense_forward([spec], seq[8])[0][1])
    a.close(); b.close()


def test_fc_chunk_host_entry_point():
    rrm = _rrm()
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=6, rho=0.05, seed=28)
    layer = rrm.layer_from_spec(spec)
    xin = torch.from_numpy(seq).pin_memory()
    out = torch.empty((6, 1, 4096, 1, 1), dtype=torch.int32).pin_memory()
    layer.step_seq_host(xin, out, 6)
    for t in range(6):
        np.testing.assert_array_equal(out[t].numpy(), orc.dense_forward([spec], seq[t])[0][1])
    layer.close()


def test_fc_chunk_host_entry_point_pipelined():
    """Chunks queued without waiting (copies and kernels of consecutive calls overlap) deliver the same outputs;
    every call has host buffers of its own, and the staging slots are reused from the third call on."""
    rrm = _rrm()
    spec = wl.fc6_i8(c_in=2048, c_out=1024)[0]
    seq = wl.fc_run_sequence(frames=31, c_in=2048, rho=0.05, seed=31, n=2)
    layer = rrm.layer_from_spec(spec, n=2)
    chunks = [(0, 4), (4, 4), (8, 8), (16, 3), (19, 12)]          # a larger T than before grows the slots mid-way
    ins = [torch.from_numpy(seq[a:a + T]).pin_memory() for a, T in chunks]
    outs = [torch.empty((T, 2, 1024, 1, 1), dtype=torch.int32).pin_memory() for _, T in chunks]
    for (a, T), x, y in zip(chunks, ins, outs):
        layer.step_seq_host_async(x, y, T)
    layer.host_sync()
    for (a, T), y in zip(chunks, outs):
        for i in range(T):
            np.testing.assert_array_equal(y[i].numpy(), orc.dense_forward([spec], seq[a + i])[0][1], err_msg=f"frame {a + i}")
    # the state is that of the last frame: a synchronous step from it is exact
    Y = layer.new_output()
    layer.step(dev(seq[30]), Y)
    np.testing.assert_array_equal(Y.cpu().numpy(), orc.dense_forward([spec], seq[30])[0][1])
    layer.close()


def test_fc6_chunk_longer_than_one_launch_holds():
    """40 frames exceed what one launch's closing sum keeps per thread: the call goes out in pieces."""
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=41, rho=0.01, seed=29)
    _run_chunks(spec, seq, 1, [40])


def test_fc6_dense_chunks_take_over_at_high_measured_density():
    """At 20 % density the second chunk on is evaluated densely on the tensor cores (the previous chunk's
    measured density decides); outputs, state and counters stay those of the delta recurrence."""
    rrm = _rrm()
    spec = wl.fc6_i8()[0]
    seq = wl.fc_run_sequence(frames=33, rho=0.20, seed=30)
    layer = rrm.layer_from_spec(spec)
    rec = orc.Recurrence([spec])
    frames = dev(seq)
    variants = []
    t0 = 0
    for T in (8, 8, 8, 8):
        Y = layer.new_output(frames=T)
        layer.step_seq(frames[t0:t0 + T], Y, T)
        nnz = 0
        for i in range(T):
            want = orc.dense_forward([spec], seq[t0 + i])[0][1]
            np.testing.assert_array_equal(Y[i].cpu().numpy().astype(np.int64), want.astype(np.int64))
            rec.step(seq[t0 + i])
            nnz += rec.nnz[0]
        st = layer.stats(0)                       # synchronises: the counters of this chunk are read back by the next call
        assert st["nnz_elems"] == nnz and st["active_macs"] == nnz * 4096
        variants.append(st["variant"])
        t0 += T
    assert variants[0] == 1 and variants[-1] == 3, variants      # gather first, dense once the density is known
    Y1 = layer.new_output()
    layer.step(frames[32], Y1)                    # the state after dense chunks is the recurrence's state
    np.testing.assert_array_equal(Y1.cpu().numpy(), orc.dense_forward([spec], seq[32])[0][1])
    layer.close()


# ------------------------------------------------------------------ few-row dense FC on the tensor cores
@pytest.mark.parametrize("c_in,c_out,shift,act,n,T", [
    (9216, 4096, -1, "none", 1, 1),       # one row: the keyframe / rrm_dense of the fc6 shape
    (9216, 4096, -1, "none", 1, 32),      # one full launch
    (9216, 4096, -1, "none", 3, 17),      # 51 rows: two launches, the state rows straddle nothing
    (9216, 4096, -1, "none", 5, 7),       # 35 rows: the last frame's rows straddle the two launches
    (4096, 1008, 7, "relu", 2, 9),        # outputs not a multiple of 128, int8 outputs through f
    (4096, 1000, 7, "relu", 2, 9),        # outputs not a multiple of 16: the general layer path, frame by frame
    (160, 528, 6, "relu", 3, 5),          # K smaller than one share per SM, ragged tiles
    (2048, 1024, -1, "none", 4, 16),      # 64 rows in one launch
    (1024, 256, -1, "none", 8, 25),       # 200 rows: two launches of 100 (112 accumulator columns), clusters of 8 K shares
    (512, 256, -1, "none", 16, 24),       # 384 rows: three launches of 128
    (256, 128, -1, "none", 150, 2),       # 300 rows in three launches: the last frame's rows straddle two of them
    (4096, 128, 5, "relu", 2, 6),         # one output block, 32 K shares: partial sums through the global scratch
    (128, 256, -1, "none", 2, 5),         # a single K slab: no split, outputs straight from the accumulators
])
def test_fc_dense_few_rows_on_tensor_cores(c_in, c_out, shift, act, n, T):
    """Dense chunks (stateless and keyframe-like) equal Eq. 3 row by row; the state after a stateful dense
    evaluation is that of the last frame, so a delta step from it is exact."""
    rrm = _rrm()
    rng = np.random.default_rng(c_in + c_out + n + T)
    spec = LayerSpec("fc", "i8", c_in, 1, 1, c_out, act=act, shift=shift, src=0)
    spec.weight = rng.integers(-127, 128, size=(c_out, c_in, 1, 1)).astype(np.int8)
    spec.bias = rng.integers(-500, 501, size=c_out).astype(np.int32)
    seq = wl.fc_run_sequence(frames=T + 1, c_in=c_in, rho=0.3, run=8, seed=c_in + T, n=n)
    layer = rrm.layer_from_spec(spec, n=n)
    frames = dev(seq)
    want = [orc.dense_forward([spec], seq[t]) for t in range(T + 1)]
    # stateless dense chunk, twice (the scratch accumulators must come back zeroed)
    for _ in range(2):
        Y = layer.new_output(frames=T)
        layer.dense_seq(frames[:T], Y, T)
        for t in range(T):
            np.testing.assert_array_equal(Y[t].cpu().numpy().astype(np.int64), want[t][0][1].astype(np.int64), err_msg=f"frame {t}")
    # a chunk dense enough to be evaluated densely with state: first chunk measures, second one switches
    Y = layer.new_output(frames=T)
    layer.step_seq(frames[:T], Y, T)
    layer.stats(0)
    layer.step_seq(frames[:T], Y, T)
    for t in range(T):
        np.testing.assert_array_equal(Y[t].cpu().numpy().astype(np.int64), want[t][0][1].astype(np.int64), err_msg=f"frame {t}")
    np.testing.assert_array_equal(layer.projection(0).cpu().numpy().astype(np.int64), want[T - 1][1][0])
    Y1 = layer.new_output()
    layer.step(frames[T], Y1)
    np.testing.assert_array_equal(Y1.cpu().numpy().astype(np.int64), want[T][0][1].astype(np.int64))
    # keyframe + dense of single frames
    layer.keyframe(frames[0], Y1)
    np.testing.assert_array_equal(Y1.cpu().numpy().astype(np.int64), want[0][0][1].astype(np.int64))
    layer.step(frames[1], Y1)
    np.testing.assert_array_equal(Y1.cpu().numpy().astype(np.int64), want[1][0][1].astype(np.int64))
    assert layer.stats(0)["error_word"] == 0
    layer.close()


# ------------------------------------------------------------------ weight-sparse x delta-sparse (Sec. 3.5 / 4.3)
@pytest.mark.parametrize("rho", [0.01, 0.05, 0.20])
def test_weight_sparse_fc_is_bit_exact_at_every_density(rho):
    """A magnitude-pruned layer (10 % of the weights kept) in the weight-sparse form: chunks, single frames, the
    keyframe and the stateless dense path all give the integers of the dense FC definition on the pruned matrix;
    the counters are those of Algorithm 1 (Table 1 counts whole columns)."""
    import paper_1802_09723_b200 as rrm
    c_in, c_out, n, F = 2048, 1040, 2, 12                     # two full 512-output slices and a ragged third
    spec = wl.fc6_i8_pruned(c_in=c_in, c_out=c_out, keep=0.10)[0]
    assert 0.08 < float(np.mean(spec.weight != 0)) < 0.12
    seq = wl.fc_run_sequence(frames=F, c_in=c_in, rho=rho, seed=61, n=n)
    seq[5] = seq[4]                                            # a frame with nothing to do
    layer = rrm.layer_from_spec(spec, n=n, variant="sparse_w")
    frames = dev(seq)
    want = [orc.dense_forward([spec], seq[t])[1][0].reshape(n, c_out) for t in range(F)]
    Y = layer.new_output(frames=4)
    t0 = 0
    for T in (4, 4, 1, 3):
        layer.step_seq(frames[t0:t0 + T], Y[:T], T)
        for i in range(T):
            np.testing.assert_array_equal(Y[i].cpu().numpy().astype(np.int64).reshape(n, c_out), want[t0 + i], err_msg=f"frame {t0 + i}")
        st = layer.stats(0)
        nnz = sum(int(np.count_nonzero(seq[t] != (seq[t - 1] if t else np.zeros_like(seq[0])))) for t in range(t0, t0 + T))
        assert st["variant"] == 4 and st["nnz_elems"] == nnz and st["active_macs"] == nnz * c_out and st["error_word"] == 0, st
        t0 += T
    np.testing.assert_array_equal(layer.projection(0).cpu().numpy().astype(np.int64).reshape(n, c_out), want[t0 - 1])
    # frame-by-frame stepping, a keyframe, and the stateless dense path on the same weights
    y1 = layer.new_output()
    layer.keyframe(frames[2], y1)
    np.testing.assert_array_equal(y1.cpu().numpy().astype(np.int64).reshape(n, c_out), want[2])
    for t in (3, 4, 5):
        layer.step(frames[t], y1)
        np.testing.assert_array_equal(y1.cpu().numpy().astype(np.int64).reshape(n, c_out), want[t])
    layer.dense(frames[9], y1)
    np.testing.assert_array_equal(y1.cpu().numpy().astype(np.int64).reshape(n, c_out), want[9])
    layer.step(frames[6], y1)                                  # the state was left alone by the dense path
    np.testing.assert_array_equal(y1.cpu().numpy().astype(np.int64).reshape(n, c_out), want[6])
    layer.close()


def test_weight_sparse_fc_full_range_deltas_and_unpruned_weights():
    """The form does not depend on the matrix being sparse (a dense matrix packs every group) and takes deltas
    outside the int8 range like the column gather does."""
    import paper_1802_09723_b200 as rrm
    c_in, c_out = 512, 512
    spec = wl.fc6_i8(c_in=c_in, c_out=c_out)[0]
    rng = np.random.default_rng(3)
    seq = rng.integers(-127, 128, size=(4, 1, c_in)).astype(np.int8)
    seq[2, 0, ::2] = seq[1, 0, ::2]
    layer = rrm.layer_from_spec(spec, variant="sparse_w")
    Y = layer.new_output(frames=4)
    layer.step_seq(dev(seq), Y, 4)
    for t in range(4):
        np.testing.assert_array_equal(Y[t].cpu().numpy().astype(np.int64).reshape(1, c_out),
                                      orc.dense_forward([spec], seq[t])[1][0].reshape(1, c_out))
    layer.close()
    # the variant exists for a lone int8 FC layer only
    conv = wl.single_conv_f32(c_in=4, c_out=4, hw=8)
    with pytest.raises(rrm.RRMError):
        rrm.net_from_specs(conv, variant="sparse_w")
