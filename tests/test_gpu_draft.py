"""GPU parity of svip_draft_step (through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest

import svip_testlib as tl
from paper_2411_18462_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2411_18462_b200 import Context, build
    build.build()
    c = Context(0, 1 << 14)
    yield c
    c.destroy()


def random_rows(rng, B, V, bf16):
    scale = np.exp(rng.uniform(np.log(0.1), np.log(10.0), size=(B, 1)))
    x = (rng.standard_normal((B, V)) * scale).astype(np.float32)
    if V >= 4:
        x[0, :] = 0.0                        # uniform row
        x[-1, rng.integers(0, V)] += 40.0    # near one-hot row
        x[B // 2, rng.integers(0, V, size=max(1, V // 7))] = -np.inf   # masked logits
    return W.to_bf16_bits(x) if bf16 else x


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("V", [1, 2, 7, 8, 33, 1000, 4099, 32000, 70001])
def test_small_shapes_all_cluster_sizes(ctx, oracle, V, bf16):
    rng = np.random.default_rng(1000 + V + int(bf16))
    B = 5
    logits = random_rows(rng, B, V, bf16)
    u = rng.random(B).astype(np.float32)
    ref = None
    for T in (1.0, 0.7, 0.0):
        for S in (1, 2, 3, 4, 5, 6, 7, 8, 0):
            ctx.set_cluster_size(S)
            got = tl.gpu_draft_step(ctx, logits, T, 0.3, u)
            tl.check_draft_against_oracle(oracle, logits, T, 0.3, u, got, "V=%d S=%d T=%g" % (V, S, T))
            if S == 1:
                ref = got
            else:   # integers do not depend on the launch shape (off CDF boundaries)
                assert np.array_equal(got[2], ref[2])
                if T == 0.0:
                    assert np.array_equal(got[0], ref[0])
    ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


@pytest.mark.parametrize("bf16", [False, True])
def test_unaligned_rows_and_strides(ctx, oracle, bf16):
    rng = np.random.default_rng(77 + int(bf16))
    for V, pad, stride in ((1001, 1, 1003), (4099, 3, 4099), (517, 5, 600), (64, 7, 71)):
        logits = random_rows(rng, 4, V, bf16)
        u = rng.random(4).astype(np.float32)
        for S in (1, 4):
            ctx.set_cluster_size(S)
            got = tl.gpu_draft_step(ctx, logits, 1.0, 0.3, u, pad_elems=pad, row_stride=stride)
            tl.check_draft_against_oracle(oracle, logits, 1.0, 0.3, u, got, "V=%d pad=%d" % (V, pad))
            got = tl.gpu_draft_step(ctx, logits, 0.0, 0.3, None, pad_elems=pad, row_stride=stride)
            tl.check_draft_against_oracle(oracle, logits, 0.0, 0.3, None, got, "greedy V=%d pad=%d" % (V, pad))
    ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


def test_closed_forms_and_stop_threshold(ctx):
    """Uniform rows give ln V and stop; one-hot rows give 0 and continue; argmax ties take the lowest index."""
    for V in (32000, 152064, 256000):
        x = np.zeros((3, V), dtype=np.float32)
        x[1, :] = -np.inf
        x[1, V - 3] = 2.0
        x[2, [5, V // 2, V - 1]] = 9.0          # three-way tie of the maximum
        tok, H, stop, stats = tl.gpu_draft_step(ctx, x, 1.0, 0.3, np.array([0.5 + 0.25 / V, 0.9, 0.1], np.float32))
        assert abs(H[0] - np.log(V)) < 1e-4 and stop[0] == 1 and tok[0] == V // 2
        assert H[1] == 0.0 and stop[1] == 0 and tok[1] == V - 3
        assert stats[0, 0] == 0.0 and abs(stats[0, 1] - V) < 1e-3 * V and stats[1, 1] == 1.0
        tok, H, stop, _ = tl.gpu_draft_step(ctx, W.to_bf16_bits(x), 0.0, 0.3, None)
        assert tok.tolist() == [0, V - 3, 5]
    assert ctx.read_status() == 0


def special_rows(V, bf16):
    """Rows that leave the fast path of the streaming loop: a steep ramp (the reference of the
    exponentials has to move many times), a late spike and a late cliff (the running sums overflow
    between two checks), rows that start with masked logits, a NaN, and huge but finite logits."""
    i = np.arange(V, dtype=np.float64)
    rows = [
        -300.0 + 600.0 * i / max(V - 1, 1),                 # ramp up
        300.0 - 600.0 * i / max(V - 1, 1),                  # ramp down
        np.where(i == V - 3, 400.0, np.sin(i)),             # spike far above everything, near the end
        np.where(i >= V // 2, 250.0 + np.cos(i), -250.0),   # cliff in the middle
        np.where(i < min(V // 3 + 1, 3000), -np.inf, np.cos(i) * 3),   # starts with masked logits
        np.where(i % 97 == 5, -np.inf, np.sin(i) * 5),      # masked logits everywhere
        np.sin(i) * 2.0,                                     # gets a NaN below
        np.cos(i) * 1.0e4,                                   # huge spread
    ]
    x = np.stack(rows).astype(np.float32)
    x[6, V // 2] = np.nan
    return W.to_bf16_bits(x) if bf16 else x


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("V", [9000, 152064])
def test_rows_off_the_fast_path(ctx, oracle, V, bf16):
    logits = special_rows(V, bf16)
    B = logits.shape[0]
    u = np.linspace(0.05, 0.95, B).astype(np.float32)
    # the oracle treats NaN like the library: as a masked logit
    clean = logits.copy()
    if bf16:
        clean[6, V // 2] = 0xFF80
    else:
        clean[6, V // 2] = -np.inf
    for T in (1.0, 0.25, 0.0):
        for S in (0, 1, 3, 8):
            ctx.set_cluster_size(S)
            got = tl.gpu_draft_step(ctx, logits, T, 0.3, u)
            tl.check_draft_against_oracle(oracle, clean, T, 0.3, u, got, "special V=%d S=%d T=%g" % (V, S, T))
    ctx.set_cluster_size(0)
    assert ctx.read_status() == 0


def test_uniform_extremes(ctx, oracle):
    """u = 0 picks the first token with mass; u just below 1 picks the last one."""
    rng = np.random.default_rng(5)
    V = 5000
    x = (rng.standard_normal((2, V)) * 2).astype(np.float32)
    x[:, :3] = -np.inf
    x[:, -2:] = -np.inf
    for u in (0.0, 1.0 - 2.0 ** -24):
        uu = np.full(2, u, dtype=np.float32)
        got = tl.gpu_draft_step(ctx, x, 1.0, 0.3, uu)
        tl.check_draft_against_oracle(oracle, x, 1.0, 0.3, uu, got, "u=%g" % u)
        assert np.all(got[0] >= 3) and np.all(got[0] < V - 2)


def test_status_word_reports_nonfinite_rows(ctx):
    x = np.zeros((2, 100), dtype=np.float32)
    x[1, :] = -np.inf
    tl.gpu_draft_step(ctx, x, 1.0, 0.3, np.zeros(2, np.float32))
    assert ctx.read_status() & 1
    assert ctx.read_status() == 0
    x[1, 4] = np.inf
    tl.gpu_draft_step(ctx, x, 1.0, 0.3, np.zeros(2, np.float32))
    assert ctx.read_status() & 1


def test_empty_batch_and_bad_arguments(ctx):
    import torch
    from paper_2411_18462_b200 import SvipError
    t = torch.zeros(16, device="cuda")
    i = torch.zeros(4, dtype=torch.int32, device="cuda")
    s = torch.zeros(4, dtype=torch.uint8, device="cuda")
    before = ctx.launch_count()
    ctx.draft_step(t, 0, 0, 16, 16, 1.0, 0.3, t, i, t, s)          # B = 0: nothing to do
    assert ctx.launch_count() == before
    for kwargs in (dict(V=0), dict(T=-1.0), dict(thresh=float("nan")), dict(dtype=7), dict(uniforms=None)):
        a = dict(logits=t, dtype=0, B=1, V=16, row_stride=16, T=1.0, thresh=0.3, uniforms=t, token=i, entropy=t,
                 stop=s)
        a.update(kwargs)
        with pytest.raises(SvipError):
            ctx.draft_step(**a)
    with pytest.raises(SvipError):   # fp32 logits must be 4-byte aligned
        ctx.draft_step(t.data_ptr() + 2, 0, 1, 8, 8, 1.0, 0.3, t, i, t, s)


@pytest.mark.parametrize("name", ["tiny", "chat", "reasoning", "ragged", "stress"])
def test_published_configs(ctx, oracle, name):
    """All draft rows of each published configuration, at full size, in the automatic launch shape."""
    w = W.make_workload(name)
    temps = {"tiny": (1.0,), "chat": (1.0, 0.0), "reasoning": (0.7,), "ragged": (1.0,), "stress": (1.0, 0.0)}[name]
    for T in temps:
        got = tl.gpu_draft_step(ctx, w.q_logits, T, w.h, w.draft_uniforms)
        c = tl.check_draft_against_oracle(oracle, w.q_logits, T, w.h, w.draft_uniforms, got, "%s T=%g" % (name, T),
                                          threads=16)
        print("draft parity", name, "T=%g" % T, c)
    assert ctx.read_status() == 0
