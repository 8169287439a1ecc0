"""svip_verify_noalloc: the verify round for callers that cannot allocate device memory.

Serving frameworks freeze their memory pool while they record or replay a fixed memory plan, some
plugins get a stream but no allocator, and some processes hand out all device memory at start-up;
such callers can neither cudaMalloc nor create an svip context (creating one allocates its
workspace).  The entry point under test takes no context and keeps its workspace in a fixed array
inside the library.  Here it must agree with svip_verify -- same accept counts and same next
tokens, bit for bit, since both run the same kernels on the same inputs -- on two calls in a row
(the second call reuses the array that the first one filled), agree with the fp64 oracle within the
tolerances of the other parity tests, and refuse more rows than the array holds.  This file sorts last so that a run stopping at the first failure has run everything else.
"""
import numpy as np
import pytest

import svip_testlib as tl

pytestmark = pytest.mark.gpu


def _case(rng, B, V, K_max, bf16):
    from paper_2411_18462_b200 import workloads as W
    lens = rng.integers(1, K_max + 1, size=B).astype(np.int32)
    cu = np.concatenate([[0], np.cumsum(lens + 1)]).astype(np.int32)
    Rp = int(cu[-1]); Rq = Rp - B
    base = (rng.standard_normal((Rp, V)) * 2.0).astype(np.float32)
    tgt = base + (rng.standard_normal((Rp, V)) * 0.4).astype(np.float32)
    q = np.empty((Rq, V), np.float32)
    for i in range(B):
        q[cu[i] - i: cu[i] - i + lens[i]] = base[cu[i]: cu[i] + lens[i]]
    tokens = rng.integers(0, V, size=Rq).astype(np.int32)
    # make most draft tokens plausible: the draft row's own argmax
    likely = q.argmax(axis=1).astype(np.int32)
    tokens = np.where(rng.random(Rq) < 0.8, likely, tokens).astype(np.int32)
    if bf16:
        q = W.to_bf16_bits(q); tgt = W.to_bf16_bits(tgt)
    return lens, cu, q, tgt, tokens, rng.random(Rp).astype(np.float32)


def test_noalloc_matches_verify_on_two_calls_in_a_row(oracle):
    import torch
    from paper_2411_18462_b200 import Context, build, verify_noalloc, SvipError
    build.build()
    dev = lambda a: torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()
    ctx = Context(0, 4096)
    rng = np.random.default_rng(2024)
    # two different rounds, back to back, the second smaller than the first so that stale
    # contents of the shared array would show
    for B, V, K_max, bf16, T in ((24, 9000, 7, True, 1.0), (5, 4099, 3, False, 0.7), (9, 1000, 4, True, 0.0)):
        lens, cu, q, tgt, tokens, u = _case(rng, B, V, K_max, bf16)
        Rp = int(cu[-1])
        # accept draws off the decision boundary (oracle values), as in the other parity tests
        u, _ = tl.guard_accept_uniforms(oracle, tokens, q, tgt, cu, T, u)
        d_tok, d_q, d_t, d_cu, d_u = dev(tokens), dev(q), dev(tgt), dev(cu), dev(u)
        out = [torch.full((B,), -5, dtype=torch.int32, device="cuda") for _ in range(4)]
        status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
        dt = 1 if bf16 else 0
        ctx.verify(d_tok, d_q, V, None, -1, 0, d_t, V, dt, d_cu, B, K_max, Rp, V, T, d_u, out[0], out[1])
        verify_noalloc(0, d_tok, d_q, V, None, -1, 0, d_t, V, dt, d_cu, B, K_max, Rp, V, T, d_u, out[2], out[3],
                       status)
        torch.cuda.synchronize()
        assert torch.equal(out[0], out[2]), (out[0], out[2])
        assert torch.equal(out[1], out[3]), (out[1], out[3])
        assert int(out[0].min()) >= 0 and int(status.item()) == 0
        # once more with no status pointer: same answer from the reused array
        out[2].fill_(-5); out[3].fill_(-5)
        verify_noalloc(0, d_tok, d_q, V, None, -1, 0, d_t, V, dt, d_cu, B, K_max, Rp, V, T, d_u, out[2], out[3])
        torch.cuda.synchronize()
        assert torch.equal(out[0], out[2]) and torch.equal(out[1], out[3])
        # and against the oracle, like svip_verify itself
        tl.check_verify_against_oracle(oracle, tokens, q, tgt, cu, T, u, (out[2].cpu().numpy(), out[3].cpu().numpy()),
                                       "noalloc B=%d V=%d T=%g" % (B, V, T))
    # more rows than the fixed array holds: a clear error, nothing launched
    with pytest.raises(SvipError) as e:
        verify_noalloc(0, d_tok, d_q, V, None, -1, 0, d_t, V, dt, None, 8193, 1, 2 * 8193, V, 1.0, d_u, out[2], out[3])
    assert e.value.code == -3
    ctx.destroy()
