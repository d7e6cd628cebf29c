"""Failure paths in the forms that cannot harm a GPU: a bounded device-side wait that runs out (the kernel returns
with an error word, the context stays usable) and a host-side deadline that runs out behind a delay of fixed length
(the call returns a status, the model recovers).  Nothing here waits without a limit and nothing faults."""
import numpy as np
import pytest

import tpi_synth as S
from tests.helpers import gpu_session, rel_l2

pytestmark = pytest.mark.gpu


def test_a_device_wait_that_runs_out_returns_an_error_word_and_the_context_stays_usable():
    """The tensor-core GEMM with its loader switched off: no operand ever arrives, every wait runs out after a few
    thousand polls, the kernel returns by itself, stores nothing, frees its tensor memory and reports code 3.  The
    very next ordinary launch of the same kernel (which needs that tensor memory) gives the right product."""
    import torch
    import paper_2410_00531_b200.ops as K
    rng = np.random.default_rng(5)
    Tn, Kd, n_out = 128, 1024, 1536
    A = torch.from_numpy(S.f32_to_bf16_bits(rng.standard_normal((Tn, Kd)).astype(np.float32)).reshape(Tn, Kd).view(np.int16)).cuda()
    W = torch.from_numpy(S.f32_to_bf16_bits((rng.standard_normal((n_out, Kd)) * 0.02).astype(np.float32)).reshape(n_out, Kd).view(np.int16)).cuda()
    Y = torch.full((Tn, n_out), 7.0, dtype=torch.float32, device="cuda")
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    K.gemm_bf16_starved(A.data_ptr(), Kd, W.data_ptr(), Y.data_ptr(), n_out, Tn, n_out, Kd, 4096, err.data_ptr())
    t1.record()
    torch.cuda.synchronize()                                     # returns: the kernel ended by itself
    assert int(err[0]) == 3                                      # DEVERR_WAIT_TIMEOUT
    assert t0.elapsed_time(t1) < 200.0                           # milliseconds, not the default quarter second per wait
    assert bool((Y == 7.0).all())                                # nothing was stored
    err.zero_()
    for _ in range(3):                                           # tensor memory was released: ordinary launches work
        K.gemm_bf16(A.data_ptr(), Kd, 0, W.data_ptr(), n_out, Y.data_ptr(), Tn * n_out, n_out, Tn, n_out, Kd, 1, err.data_ptr())
    torch.cuda.synchronize()
    assert int(err[0]) == 0
    want = S.as_f64(A.cpu().numpy().view(np.uint16)) @ S.as_f64(W.cpu().numpy().view(np.uint16)).T
    assert rel_l2(Y.cpu().numpy(), want) < 2e-5


@pytest.mark.parametrize("window", [0, 2])
def test_host_deadline_runs_out_and_the_model_recovers(window):
    """TPI_ERR_TIMEOUT: a delay of fixed length (a spin kernel with a fixed cycle count, ~0.4 s) sits ahead of the step
    on the model's own compute stream and the deadline is cut to 50 ms.  The call gives up with the timeout status and
    leaves the host position alone; further steps are refused until the caller re-synchronises; after tpi_reset
    (which drains the stream) the prompt pass and the decode steps give the tokens they gave before."""
    import torch
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C1"].with_(n_layers=4)
    toks = S.prompt_tokens(shape)
    with gpu_session(shape, 64, 16, 2, window) as ses:
        t0, lg0 = P.prefill(ses.h, toks, shape.vocab)
        seq0 = P.decode_run(ses.h, t0, 5)
        P.reset(ses.h)
        t0b, _ = P.prefill(ses.h, toks, 0)
        assert t0b == t0
        P.set_option(ses.h, P.OPT_WAIT_DEADLINE_MS, 50)
        with torch.cuda.stream(ses.compute):
            torch.cuda._sleep(int(0.4 * 1.9e9))                  # fixed cycle count; ends by itself
        with pytest.raises(P.TpiError) as e:
            P.decode_step(ses.h, t0, 0)
        assert e.value.code == -7                                # TPI_ERR_TIMEOUT
        assert P.position(ses.h) == len(toks)                    # the host position did not move
        with pytest.raises(P.TpiError) as e:
            P.decode_step(ses.h, t0, 0)                          # refused until re-synchronised
        assert e.value.code == -9
        P.set_option(ses.h, P.OPT_WAIT_DEADLINE_MS, 60000)
        P.reset(ses.h)                                           # drains the stream, position 0 on both sides
        t1, lg1 = P.prefill(ses.h, toks, shape.vocab)
        seq1 = P.decode_run(ses.h, t1, 5)
        assert t1 == t0 and np.array_equal(lg1, lg0) and (seq1 == seq0).all()
        with pytest.raises(P.TpiError):
            P.set_option(ses.h, P.OPT_WAIT_DEADLINE_MS, 0)


def test_a_rejected_token_leaves_position_and_window_consistent():
    """A step that the device rejects (token id out of range, found by the embedding kernel's self-check when ids are
    chained on the device is not reachable from the host API, so the host check stands in) must not move the position,
    and a streamed model must keep working afterwards with the same results."""
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C1"].with_(n_layers=3)
    toks = S.prompt_tokens(shape)
    with gpu_session(shape, 64, 16, 2, 2) as ses:
        t0, _ = P.prefill(ses.h, toks, 0)
        ref = P.decode_run(ses.h, t0, 4)
        P.set_position(ses.h, len(toks))
        with pytest.raises(P.TpiError) as e:
            P.decode_step(ses.h, shape.vocab + 5, 0)
        assert e.value.code == -5 and P.position(ses.h) == len(toks)
        again = P.decode_run(ses.h, t0, 4)
        assert (again == ref).all()


def test_guard_zones_catch_a_write_past_a_buffer(monkeypatch):
    """TPI_DEBUG=1: guard zones after every arena buffer.  A clean run raises no alarm (same tokens as without the
    zones); one byte written into the zone behind the first buffer (the embedding table) makes the next call
    return TPI_ERR_DEVICE_CHECK naming zone 0; with the byte put back the model carries on."""
    import torch
    import paper_2410_00531_b200 as P
    shape = S.CONFIGS["C1"]
    toks = S.prompt_tokens(shape)
    monkeypatch.delenv("TPI_DEBUG", raising=False)
    with gpu_session(shape, 64, 16, 2) as ses:
        plain_bytes = ses.dev.numel()
        t_ref, _ = P.prefill(ses.h, toks, 0)
        seq_ref = P.decode_run(ses.h, t_ref, 4)
    monkeypatch.setenv("TPI_DEBUG", "1")
    for window in (0, 2):
        with gpu_session(shape, 64, 16, 2, window) as ses:
            if window == 0:
                assert ses.dev.numel() > plain_bytes                 # the zones take room
            t0, _ = P.prefill(ses.h, toks, 0)
            seq = P.decode_run(ses.h, t0, 4)
            assert t0 == t_ref and (seq == seq_ref).all()            # no false alarm, same results
            zone0 = (shape.vocab * shape.hidden * 4 + 255) // 256 * 256
            old = int(ses.dev[zone0 + 17])
            ses.dev[zone0 + 17] = old ^ 0x5A
            torch.cuda.synchronize()
            with pytest.raises(P.TpiError) as e:
                P.decode_step(ses.h, int(seq[-1]), 0)
            assert e.value.code == -8 and "guard zone 0" in str(e.value)
            assert P.position(ses.h) == len(toks) + 4                # a rejected step does not move the position
            ses.dev[zone0 + 17] = old
            torch.cuda.synchronize()
            tok, _ = P.decode_step(ses.h, int(seq[-1]), 0)
            P.set_position(ses.h, len(toks) + 4)
            tok2, _ = P.decode_step(ses.h, int(seq[-1]), 0)
            assert tok == tok2
