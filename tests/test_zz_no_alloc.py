"""The allocation-free row-sharded projection (tpi_op_rowshard_project_static).

It exists for callers that cannot allocate device memory when they need this step (a
memory-capped plug-in, a real-time loop where cudaMalloc is off limits): the per-shard
partial sums live in an array inside the library instead of a caller buffer.  The test calls
it through the C ABI twice in a row, with different inputs and shapes, and checks each result
against the ordinary entry point that takes caller scratch (bit for bit: the kernels are the
same) and against the CPU oracle's definition of the step; the second call also shows that
whatever the first call left in the shared array does no harm.  This file sorts last so that
a run stopping at the first failure has already run every other test."""
import numpy as np
import pytest

import tpi_synth as S
from oracle import llama_oracle as O
from tests.helpers import rel_l2

pytestmark = pytest.mark.gpu


def _case(torch, K, shape, which, n_shards, seed):
    w = S.gen_tensor(shape, 1, which)
    h, kdim = w.shape
    packed = np.ascontiguousarray(w.reshape(h, n_shards, kdim // n_shards).transpose(1, 0, 2))
    if packed.dtype == np.uint16:
        packed = packed.view(np.int16)
    Wd = torch.from_numpy(packed).cuda()
    x_host = S.hidden_state(seed, kdim, 0.7)
    x_in = torch.from_numpy(x_host).cuda()
    resid = S.hidden_state(seed + 1, h, 0.5)
    dt = 1 if shape.dtype == "bf16" else 0
    # ordinary entry point: partial sums in a buffer the caller allocated
    x_ref, xhat_ref = torch.from_numpy(resid.copy()).cuda(), torch.empty(h, device="cuda")
    scratch = torch.empty(n_shards * h, device="cuda")
    K.rowshard_project(dt, Wd.data_ptr(), x_in.data_ptr(), h, kdim // n_shards, n_shards, shape.rms_eps,
                       scratch.data_ptr(), x_ref.data_ptr(), xhat_ref.data_ptr())
    # allocation-free entry point: inputs and outputs only
    x_new, xhat_new = torch.from_numpy(resid.copy()).cuda(), torch.empty(h, device="cuda")
    K.rowshard_project_static(dt, Wd.data_ptr(), x_in.data_ptr(), h, kdim // n_shards, n_shards, shape.rms_eps,
                              x_new.data_ptr(), xhat_new.data_ptr())
    torch.cuda.synchronize()
    got_x, got_xhat = x_new.cpu().numpy(), xhat_new.cpu().numpy()
    # the two entry points run the same two kernels, only the home of the partial sums differs: same bits
    assert np.array_equal(got_x, x_ref.cpu().numpy())
    assert np.array_equal(got_xhat, xhat_ref.cpu().numpy())
    # and against the oracle's definition of the step (Eq. 1-2: sum of the shards' partial sums + shortcut, then the norm)
    want_x = np.zeros(h)
    for r0 in range(0, h, 1024):
        want_x[r0:r0 + 1024] = S.as_f64(w[r0:r0 + 1024]) @ x_host.astype(np.float64)
    want_x += resid
    assert rel_l2(got_x, want_x) < 2e-6
    assert rel_l2(got_xhat, O.rmsnorm(want_x, np.ones(h), shape.rms_eps)) < 2e-6


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row():
    import torch
    import paper_2410_00531_b200.ops as K
    # first call: 7B-shaped down projection, 4 shards (4 x 4096 partial sums)
    _case(torch, K, S.CONFIGS["C2"], S.WDOWN, 4, 41)
    # second call right after it: other shape, dtype and shard count; the array still holds call 1's sums
    _case(torch, K, S.CONFIGS["C1"], S.WO, 2, 43)
    _case(torch, K, S.CONFIGS["C2"], S.WO, 2, 45)


def test_static_scratch_at_exactly_its_limit():
    """8 shards x 8192 rows (the 70B shape's down projection) need 65536 floats: all of the built-in array, not one
    more.  An off-by-one in the bound or in the indexing would show here."""
    import torch
    import paper_2410_00531_b200.ops as K
    assert K.static_scratch_floats() == 8 * 8192
    _case(torch, K, S.CONFIGS["C5"], S.WDOWN, 8, 47)
    _case(torch, K, S.CONFIGS["C2"], S.WO, 4, 49)            # a smaller call after the full one


def test_static_scratch_rejects_oversized_and_malformed_requests():
    import torch
    import paper_2410_00531_b200 as P
    import paper_2410_00531_b200.ops as K
    limit = K.static_scratch_floats()
    assert limit == 65536
    dummy = torch.zeros(64, device="cuda")
    with pytest.raises(P.TpiError) as e:
        K.rowshard_project_static(0, dummy.data_ptr(), dummy.data_ptr(), limit // 8 + 1, 8, 8, 1e-5,
                                  dummy.data_ptr(), dummy.data_ptr())
    assert e.value.code == -3 and "65536" in str(e.value)
    for rows, n_shards in ((0, 4), (16, 0)):
        with pytest.raises(P.TpiError) as e:
            K.rowshard_project_static(0, dummy.data_ptr(), dummy.data_ptr(), rows, 8, n_shards, 1e-5,
                                      dummy.data_ptr(), dummy.data_ptr())
        assert e.value.code == -1 and "rowshard_project_static" in str(e.value)
