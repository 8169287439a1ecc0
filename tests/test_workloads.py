"""The seeded workload generators: determinism, shapes, and (with the oracle) that the ragged
workload's draft lengths are exactly what the entropy stop rule of Eq. 7 produces."""
import numpy as np

from paper_2411_18462_b200 import workloads as W


def test_deterministic_and_thread_independent():
    a = W.make_workload("chat", B=3, V=1000, threads=1)
    b = W.make_workload("chat", B=3, V=1000, threads=4)
    for f in ("q_logits", "target_logits", "draft_uniforms", "verify_uniforms", "draft_len", "cu_rows"):
        assert np.array_equal(getattr(a, f), getattr(b, f)), f
    c = W.make_workload("chat", B=3, V=1000, seed=a.seed + 1)
    assert not np.array_equal(a.q_logits, c.q_logits)


def test_shapes_and_ranges():
    for name, spec in W.SPECS.items():
        w = W.make_workload(name, B=min(spec["B"], 4), V=512)
        assert w.q_logits.shape == (w.n_draft_rows, 512) and w.target_logits.shape == (w.n_target_rows, 512)
        assert w.q_logits.dtype == (np.uint16 if spec["dtype"] == "bf16" else np.float32)
        assert w.cu_rows[-1] == (w.draft_len + 1).sum()
        for u in (w.draft_uniforms, w.verify_uniforms):
            assert u.dtype == np.float32 and u.min() >= 0.0 and u.max() < 1.0
        assert np.all((w.draft_len >= 1) & (w.draft_len <= w.K_max))


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e38], dtype=np.float32)
    b = W.to_bf16_bits(x)
    back = W.bf16_bits_to_f32(b)
    # 1.00390625 = 1 + 2^-8 is a tie between 1.0 and 1.0078125: even mantissa wins (1.0)
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == np.float32(1.015625) and back[3] == -2.5


def test_tiny_plants(oracle):
    w = W.make_workload("tiny")
    tok, H, stop = oracle.draft_step(w.q_logits, w.T, w.h, w.draft_uniforms)
    for p in w.notes["onehot_pos"]:
        assert H[p] < 1e-6 and stop[p] == 0
    for p in w.notes["uniform_pos"]:
        assert abs(H[p] - np.log(w.V)) < 1e-9 and stop[p] == 1
    for p in w.notes["copied_pos"]:
        assert np.array_equal(w.q_logits[p], w.target_logits[p])


def test_ragged_lengths_follow_the_stop_rule(oracle):
    """Running the entropy rule over each sequence's draft rows stops exactly at K_i (or hits the cap)."""
    w = W.make_workload("ragged", B=10)
    tok, H, stop = oracle.draft_step(w.q_logits, w.T, w.h, w.draft_uniforms, threads=8)
    for i in range(w.B):
        r0 = int(w.cu_rows[i]) - i
        K = int(w.draft_len[i])
        flags = stop[r0:r0 + K]
        assert not flags[:-1].any()
        assert flags[-1] == 1 or K == w.K_max
        assert np.all(np.abs(np.sqrt(H[r0:r0 + K]) - w.h) > 0.01)
