"""The allocation-free delta-FC entry point against the ordinary one and against the CPU oracle.

Who needs it: callers that cannot allocate device memory - plug-ins whose host hands them a
fixed memory budget and forbids cudaMalloc afterwards, real-time loops that must not wait on the
allocator, processes under a hard GPU memory cap.  rrm_fc_step_noalloc keeps its
only working memory (the lists of non-zero delta entries) in a fixed array inside the library,
so every call shares it and it still holds the previous call's contents.  That is why this test
makes several calls in a row, with a different number of non-zeros each time: stale entries from
an earlier, longer list must never leak into a later, shorter one.

Collected last on purpose (file name), so a run that stops at the first failure has already
run everything else.  It passes alone in a fresh process as well as after the other tests."""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import rrm_oracle as orc

pytestmark = pytest.mark.gpu


def test_noalloc_entry_matches_rrm_step_on_consecutive_calls():
    import paper_1802_09723_b200 as rrm
    n, c_in, c_out = 4, 2048, 1040          # 1040 = 8 full output slices + a ragged one
    spec = wl.fc6_i8(c_in=c_in, c_out=c_out)[0]
    seq = wl.fc_run_sequence(frames=5, c_in=c_in, rho=0.20, seed=77, n=n)
    seq[2] = seq[1]                          # a call with nothing to do ...
    seq[3, :, 64:96] = 127 - seq[2, :, 64:96]   # ... then a short list after the long ones

    # ordinary entry point: the library owns state and working memory
    layer = rrm.layer_from_spec(spec, n=n)
    Y_ref = layer.new_output()

    # allocation-free entry point: the caller owns the state; every buffer exists before the first call
    Wt = torch.from_numpy(np.ascontiguousarray(spec.weight.reshape(c_out, c_in).T)).cuda()
    Xprev = torch.zeros((n, c_in), dtype=torch.int8, device="cuda")
    P = torch.from_numpy(np.tile(spec.bias, (n, 1))).cuda()
    Y = torch.empty((n, c_out), dtype=torch.int32, device="cuda")
    frames = [torch.from_numpy(seq[t]).cuda() for t in range(seq.shape[0])]
    torch.cuda.synchronize()

    for t, x in enumerate(frames):
        layer.step(x, Y_ref)
        before = torch.cuda.memory_allocated()
        status = rrm.fc_step_noalloc(Wt, x, Xprev, P, Y, n, c_in, c_out)
        assert status == 0, status
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert torch.equal(Y, Y_ref.reshape(n, c_out)), f"call {t}: output differs from rrm_step"
        # ... and directly against the CPU oracle's dense evaluation of this frame (Eq. 3), bit for bit
        want = orc.dense_forward([spec], seq[t])[1][0].reshape(n, c_out)
        assert np.array_equal(Y.cpu().numpy().astype(np.int64), want), f"call {t}: output differs from the oracle"
        assert torch.equal(P, layer.projection(0).reshape(n, c_out)), f"call {t}: projection differs"
        assert torch.equal(Xprev, x), f"call {t}: snapshot not updated in place"
    layer.close()


def test_noalloc_entry_rejects_sizes_beyond_its_fixed_array():
    import paper_1802_09723_b200 as rrm
    x = torch.zeros(64, dtype=torch.int8, device="cuda")
    p = torch.zeros(64, dtype=torch.int32, device="cuda")
    CAPACITY, SHAPE = -5, -2
    assert rrm.fc_step_noalloc(x, x, x, p, None, 17, 16, 16) == CAPACITY          # too many streams
    assert rrm.fc_step_noalloc(x, x, x, p, None, 1, 16384 + 16, 16) == CAPACITY   # input too wide
    assert rrm.fc_step_noalloc(x, x, x, p, None, 1, 24, 16) == SHAPE              # not a multiple of 16
    assert rrm.fc_step_noalloc(None, x, x, p, None, 1, 16, 16) == -1
    torch.cuda.synchronize()
