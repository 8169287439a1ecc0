"""Vocabulary-parallel draft step on one GPU: G ranks are emulated one after another on column shards
of the same rows; the result must equal the oracle's draft step on the whole rows."""
import numpy as np
import pytest

import svip_testlib as tl
from paper_2411_18462_b200 import vocab_parallel as VP
from paper_2411_18462_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2411_18462_b200 import Context, build
    build.build()
    c = Context(0, 1 << 12)
    yield c
    c.destroy()


def run_sharded(ctx, logits, G, T, h, u):
    import torch
    B, V = logits.shape
    dt = tl.dtype_code(logits)
    d = tl.to_device(logits)
    esz = logits.itemsize
    du = tl.to_device(np.asarray(u, dtype=np.float32))
    bounds = [VP.shard_bounds(V, G, r) for r in range(G)]
    partials = torch.zeros((G, B, 4), dtype=torch.float32, device="cuda")
    for r, (lo, hi) in enumerate(bounds):
        if hi > lo:
            ctx.vp_partial(d.data_ptr() + lo * esz, dt, B, hi - lo, V, T, lo, partials[r])
        else:   # an empty shard contributes nothing: maximum -inf, no mass
            partials[r, :, 0] = -np.inf
    outs = []
    tokens = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    for r, (lo, hi) in enumerate(bounds):
        ent = torch.zeros(B, device="cuda"); stop = torch.zeros(B, dtype=torch.uint8, device="cuda")
        tok = torch.zeros(B, dtype=torch.int32, device="cuda"); owner = torch.zeros(B, dtype=torch.int32, device="cuda")
        tgt = torch.zeros(B, device="cuda"); act = torch.zeros(B, dtype=torch.uint8, device="cuda")
        ctx.vp_combine(partials, G, r, B, T, h, du, ent, stop, tok, owner, tgt, act)
        if T > 0 and hi > lo:
            ctx.vp_locate(d.data_ptr() + lo * esz, dt, B, hi - lo, V, T, tgt, act, lo, tok)
        torch.cuda.synchronize()
        tokens = torch.maximum(tokens, tok)          # what the max-reduce over ranks does
        outs.append((ent.cpu().numpy(), stop.cpu().numpy(), owner.cpu().numpy(), act.cpu().numpy()))
    for o in outs[1:]:                               # every rank computed the same entropy, flags and owners
        assert np.array_equal(o[0], outs[0][0]) and np.array_equal(o[1], outs[0][1]) and np.array_equal(o[2], outs[0][2])
    if T > 0:
        assert np.array_equal(sum(o[3].astype(int) for o in outs), np.ones(B, dtype=int))   # exactly one owner per row
    return tokens.cpu().numpy(), outs[0][0], outs[0][1], None


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("V", [40, 1000, 4099, 32000])
def test_shards_match_whole_rows(ctx, oracle, V, bf16):
    rng = np.random.default_rng(300 + V + int(bf16))
    B = 6
    x = (rng.standard_normal((B, V)) * np.exp(rng.uniform(np.log(0.2), np.log(8.0), size=(B, 1)))).astype(np.float32)
    x[0, :] = 0.0
    x[1, rng.integers(0, V)] += 40.0
    x[2, : V // 2] = -np.inf                        # whole shards without mass
    logits = W.to_bf16_bits(x) if bf16 else x
    u = rng.random(B).astype(np.float32)
    for G in (1, 2, 3, 8):
        for T in (1.0, 0.5, 0.0):
            got = run_sharded(ctx, logits, G, T, 0.3, u)
            tl.check_draft_against_oracle(oracle, logits, T, 0.3, u, got, "V=%d G=%d T=%g" % (V, G, T))
    assert ctx.read_status() == 0


def test_chat_rows_eight_shards(ctx, oracle):
    w = W.make_workload("chat")
    got = run_sharded(ctx, w.q_logits, 8, w.T, w.h, w.draft_uniforms)
    c = tl.check_draft_against_oracle(oracle, w.q_logits, w.T, w.h, w.draft_uniforms, got, "chat G=8", threads=8)
    print("vocab-parallel chat", c)


def test_shard_bounds():
    for V in (1, 7, 8, 1000, 32000, 152064):
        for G in (1, 2, 3, 8, 64):
            b = [VP.shard_bounds(V, G, r) for r in range(G)]
            assert b[0][0] == 0 and b[-1][1] == V and all(x[1] == y[0] for x, y in zip(b, b[1:]))
            assert all(lo % 8 == 0 for lo, hi in b if hi > lo)
