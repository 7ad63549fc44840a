"""psmc_logits_pass_static: the logit pass for callers that cannot allocate device memory.

Such a caller (a custom-op hook inside a serving runtime that owns all device memory, a plug-in that
may not call cudaMalloc because it would stall the device, a loop with a no-allocation-after-start
rule) passes only inputs and outputs; the span partials live in a fixed array inside the library.
The test calls the entry point through the C-ABI twice in a row, on different shapes so that the
second call finds the first call's leftovers in the shared array, and checks each result against
psmc_logits_pass (caller-provided scratch) on the same inputs and, row by row, against the CPU oracle.
It is collected last on purpose.
"""
import ctypes as C

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

TOL = 1e-5  # the tolerance the parity tests use for log omega and log p(y)


def _outputs(R, dev):
    return (torch.full((R,), -7, dtype=torch.int32, device=dev), torch.zeros(R, dtype=torch.float64, device=dev),
            torch.zeros(R, dtype=torch.float64, device=dev), torch.zeros(1, dtype=torch.int32, device=dev))


def _reference(B, logits, beta, alpha_t, u, done):
    R, V = logits.shape
    nbytes = B.logits_pass_scratch_bytes(R, V)
    scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=logits.device)
    off = (-scratch.data_ptr()) % 256
    tok, logp, loginc, status = _outputs(R, logits.device)
    B.logits_pass(logits, beta, alpha_t, u, done, scratch[off: off + nbytes], tok, logp, loginc, status)
    torch.cuda.synchronize()
    return tok.cpu().numpy(), logp.cpu().numpy(), loginc.cpu().numpy(), int(status.item())


def test_static_scratch_entry_point_matches_the_scratch_taking_one_twice_in_a_row():
    from paper_2602_10273_b200 import binding as B
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = torch.Generator(device=dev).manual_seed(1234)
    cases = [  # (rows, vocab, dtype, beta, alpha_t, rows marked done)
        (24, 50000, torch.bfloat16, 4.0, 4.0, [3, 7]),
        (5, 3001, torch.float32, 2.5, 4.0, []),
    ]
    for R, V, dtype, beta, alpha_t, done_rows in cases:
        logits = (torch.randn(R, V, device=dev, generator=gen) * 3.0).to(dtype)
        u = torch.rand(R, dtype=torch.float64, device=dev, generator=gen).clamp_(1e-12, 1.0 - 1e-12)
        done = torch.zeros(R, dtype=torch.uint8, device=dev)
        if done_rows:
            done[done_rows] = 1
        assert B.logits_pass_scratch_bytes(R, V) <= B.STATIC_SCRATCH_BYTES
        tok, logp, loginc, status = _outputs(R, dev)
        B.logits_pass_static(logits, beta, alpha_t, u, done, tok, logp, loginc, status)
        torch.cuda.synchronize()
        r_tok, r_logp, r_loginc, r_status = _reference(B, logits, beta, alpha_t, u, done)
        assert int(status.item()) == r_status == B.OK
        assert np.array_equal(tok.cpu().numpy(), r_tok)
        live = np.ones(R, bool)
        live[done_rows] = False
        assert (r_tok[live] >= 0).all() and (r_tok[~live] == -7).all()       # finished rows are left untouched
        assert np.abs(logp.cpu().numpy() - r_logp).max() <= TOL
        assert np.abs(loginc.cpu().numpy() - r_loginc).max() <= TOL
        # and the oracle's row function on the same bits (tokens equal unless the uniform sits on a CDF boundary)
        import parity as P
        P.check_rows_against_oracle(logits, beta, alpha_t, u.cpu().numpy(), tok.cpu().numpy(), logp.cpu().numpy(),
                                  loginc.cpu().numpy(), rows=np.nonzero(live)[0])


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    from paper_2602_10273_b200 import binding as B
    dev = torch.device("cuda", 0)
    R, V = 300000, 1024                                    # 300000 rows x 1 span x 16 bytes > 4 MiB
    assert B.logits_pass_scratch_bytes(R, V) > B.STATIC_SCRATCH_BYTES
    dummy = torch.zeros(8, dtype=torch.float64, device=dev)
    rc = B.lib().psmc_logits_pass_static(dummy.data_ptr(), B.F32, R, V, V, 4.0, 4.0, dummy.data_ptr(), None,
                                         dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(), None)
    assert rc == B.E_TOO_LARGE                              # refused on the host: nothing was enqueued
    assert b"fixed scratch" in B.lib().psmc_strerror(rc)
    torch.cuda.synchronize()
