"""Seeded synthetic workloads: logits shaped like the paper's draft / target vocabularies.

This module only draws inputs.  It holds none of the method's arithmetic (no
softmax, entropy, acceptance or sampling) and is the one module that both the
CUDA tests and the CPU oracle tests may share.  numpy only.

The five workloads stand in for the paper's MT-Bench / MATH / AIME / GPQA runs
with Qwen2.5-, QwQ- and Vicuna-sized vocabularies (Section 3), whose data and
weights are not available: vocabulary sizes 32000 and 152064 (plus a 256000
stress case), temperature 1 and greedy decoding, threshold h = 0.3, draft
lengths up to and past the paper's cap of 40.

Every array is a function of (workload name, seed, shape overrides) only:
random streams are Philox counters keyed by (seed, tensor id, row block), so
blocks can be drawn on several threads without changing the result.

Layout of a generated workload (all numpy, host memory):
  draft_len        int32 [B]           K_i
  cu_rows          int64 [B+1]         exclusive prefix of (K_i + 1)
  q_logits         [sum K_i, V]        draft rows packed sequence after sequence
  target_logits    [sum (K_i+1), V]    target rows packed the same way
  draft_uniforms   float32 [sum K_i]   one draw per draft row (token sampling)
  verify_uniforms  float32 [sum (K_i+1)]  K_i accept draws then one sampling draw
bf16 logits are uint16 bit patterns, fp32 logits are float32.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 0x5C1B0000

SPECS = {
    #            B    V       dtype   K_max  T    h    ragged
    "tiny":      dict(B=1, V=32000, dtype="f32", K_max=8, T=1.0, h=0.3, index=0),
    "chat":      dict(B=16, V=32000, dtype="bf16", K_max=16, T=1.0, h=0.3, index=1),
    "reasoning": dict(B=32, V=152064, dtype="bf16", K_max=32, T=0.7, h=0.3, index=2),
    "ragged":    dict(B=128, V=152064, dtype="bf16", K_max=64, T=1.0, h=0.3, index=3),
    "stress":    dict(B=256, V=256000, dtype="f32", K_max=8, T=1.0, h=0.3, index=4),
}

_T_DRAFT, _T_NOISE, _T_SCALE, _T_LEN, _T_UNI_D, _T_UNI_V, _T_PLANT, _T_PERM, _T_SIGMA = range(9)
_ROW_BLOCK = 16


@dataclass
class Workload:
    name: str
    B: int
    V: int
    dtype: str          # "f32" | "bf16"
    K_max: int
    T: float
    h: float
    seed: int
    draft_len: np.ndarray
    cu_rows: np.ndarray
    q_logits: np.ndarray
    target_logits: np.ndarray
    draft_uniforms: np.ndarray
    verify_uniforms: np.ndarray
    notes: dict = field(default_factory=dict)

    @property
    def n_draft_rows(self) -> int:
        return int(self.cu_rows[-1]) - self.B

    @property
    def n_target_rows(self) -> int:
        return int(self.cu_rows[-1])

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns, round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, tensor: int, block: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) | tensor, block]))


def _uniform24(seed: int, tensor: int, n: int) -> np.ndarray:
    """n floats k / 2^24, k in [0, 2^24): exact in fp32, inside [0, 1)."""
    k = _rng(seed, tensor).integers(0, 1 << 24, size=n, dtype=np.int64)
    return (k.astype(np.float64) / float(1 << 24)).astype(np.float32)


def _store(dst: np.ndarray, lo: int, rows: np.ndarray, dtype: str):
    dst[lo:lo + rows.shape[0]] = to_bf16_bits(rows) if dtype == "bf16" else rows.astype(np.float32)


def _as_f32(rows: np.ndarray, dtype: str) -> np.ndarray:
    return bf16_bits_to_f32(rows) if dtype == "bf16" else rows


def _parallel(fn, n_blocks: int, threads: int):
    if threads <= 1 or n_blocks <= 1:
        for b in range(n_blocks):
            fn(b)
        return
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(fn, range(n_blocks)))


def _row_maps(draft_len: np.ndarray):
    """For every target row: sequence, position, and the draft row under it (-1 for the bonus row)."""
    B = draft_len.size
    cu = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(draft_len.astype(np.int64) + 1, out=cu[1:])
    seq = np.repeat(np.arange(B, dtype=np.int64), draft_len.astype(np.int64) + 1)
    pos = np.arange(cu[-1], dtype=np.int64) - cu[seq]
    drow = np.where(pos < draft_len[seq], cu[seq] - seq + pos, -1)
    return cu, seq, pos, drow


def make_workload(name: str, seed: int | None = None, B: int | None = None, V: int | None = None,
                  K_max: int | None = None, threads: int = 8) -> Workload:
    """Draws workload `name`; B, V, K_max override the published shape (same recipe, smaller case)."""
    spec = dict(SPECS[name])
    if B is not None:
        spec["B"] = B
    if V is not None:
        spec["V"] = V
    if K_max is not None:
        spec["K_max"] = K_max
    if seed is None:
        seed = BASE_SEED + spec["index"]
    B, V, K, dtype = spec["B"], spec["V"], spec["K_max"], spec["dtype"]
    notes = {}

    # ---- draft lengths
    if name == "ragged":
        draft_len = _rng(seed, _T_LEN).integers(1, K + 1, size=B, dtype=np.int64).astype(np.int32)
    else:
        draft_len = np.full(B, K, dtype=np.int32)
    cu, seq, pos, drow = _row_maps(draft_len)
    Rp = int(cu[-1])
    Rq = Rp - B
    np_dtype = np.uint16 if dtype == "bf16" else np.float32
    q = np.empty((Rq, V), dtype=np_dtype)
    t = np.empty((Rp, V), dtype=np_dtype)
    n_blocks = (Rp + _ROW_BLOCK - 1) // _ROW_BLOCK

    # ---- per-target-row parameters (one base row per target row; draft rows reuse it)
    g = _rng(seed, _T_SCALE)
    if name == "tiny":
        scale = np.full(Rp, 2.0)
        sigma = np.zeros(Rp)                # target rows are independent draws, see below
    elif name == "chat":
        scale = np.exp(g.uniform(math.log(0.1), math.log(10.0), size=Rp))
        sigma = np.full(Rp, 0.5)
    elif name == "reasoning":
        scale = np.exp(g.uniform(math.log(0.1), math.log(10.0), size=Rp))
        sigma = _rng(seed, _T_SIGMA).uniform(0.2, 2.0, size=Rp)
    elif name == "ragged":
        # heavy-tailed scale |t_3| (Student-t, nu = 3), clipped to keep bf16 logits tame
        z = g.standard_normal(Rp)
        chi = g.chisquare(3.0, size=Rp)
        scale = np.clip(np.abs(z / np.sqrt(chi / 3.0)), 0.05, 30.0)
        sigma = np.full(Rp, 0.5)
        # the row at which the entropy rule stops the draft (last draft row, unless the cap K_max
        # ended it) and the bonus row stay diffuse; every earlier row gets a dominant token
        is_last = (pos == draft_len[seq] - 1) & (draft_len[seq] < K)
        diffuse = is_last | (pos == draft_len[seq])
        scale = np.where(diffuse, np.minimum(scale, 4.0), scale)
        boost = _rng(seed, _T_PLANT).uniform(7.0, 12.0, size=Rp)
        plant_at = _rng(seed, _T_PLANT, 1).integers(0, V, size=Rp)
        notes["continue_rows"] = int((~diffuse).sum())
    elif name == "stress":
        scale = np.ones(Rp)
        sigma = np.ones(Rp)
        zipf = (-1.1 * np.log(np.arange(1, V + 1, dtype=np.float64))).astype(np.float32)
    else:
        raise KeyError(name)

    if name == "tiny":
        # K = 8 draft rows per sequence: rows 1, 4, 6 near one-hot (+30 at a random index), rows 2, 5
        # exactly uniform (all zeros).  The target copies draft rows 1 and 2 bit for bit.
        gp = _rng(seed, _T_PLANT)
        onehot_pos = [p for p in (1, 4, 6) if p < K]
        uniform_pos = [p for p in (2, 5) if p < K]
        plant_idx = gp.integers(0, V, size=(B, K))
        notes.update(onehot_pos=onehot_pos, uniform_pos=uniform_pos,
                     copied_pos=[p for p in (1, 2) if p < K])

    def block(b):
        lo, hi = b * _ROW_BLOCK, min((b + 1) * _ROW_BLOCK, Rp)
        n = hi - lo
        base = _rng(seed, _T_DRAFT, b).standard_normal((n, V), dtype=np.float32)
        noise = _rng(seed, _T_NOISE, b).standard_normal((n, V), dtype=np.float32)
        if name == "stress":
            gperm = _rng(seed, _T_PERM, b)
            for r in range(n):
                base[r] = zipf[gperm.permutation(V)]
        else:
            base *= scale[lo:hi, None].astype(np.float32)
        if name == "ragged":
            for r in range(n):
                R = lo + r
                if not diffuse[R]:
                    s = float(scale[R])
                    level = max(float(base[r].max()), math.log(V) + 0.5 * s * s)
                    base[r, plant_at[R]] = level + boost[R]
        if name == "tiny":
            for r in range(n):
                R = lo + r
                i, j = int(seq[R]), int(pos[R])
                if j in onehot_pos:
                    base[r, plant_idx[i, j]] += 30.0
                if j in uniform_pos:
                    base[r, :] = 0.0
        # the draft row is the rounded base row; the target row is rounded (draft + noise)
        d_store = to_bf16_bits(base) if dtype == "bf16" else base
        d_val = _as_f32(d_store, dtype)
        if name == "tiny":
            tgt = noise * np.float32(2.0)
            for r in range(n):
                if int(pos[lo + r]) in notes["copied_pos"]:
                    tgt[r] = d_val[r]
        else:
            tgt = d_val + noise * sigma[lo:hi, None].astype(np.float32)
        _store(t, lo, tgt, dtype)
        dr = drow[lo:hi]
        has = dr >= 0
        if has.any():
            q[dr[has]] = d_store[has]

    _parallel(block, n_blocks, threads)

    return Workload(name=name, B=B, V=V, dtype=dtype, K_max=K, T=spec["T"], h=spec["h"], seed=seed,
                    draft_len=draft_len, cu_rows=cu, q_logits=q, target_logits=t,
                    draft_uniforms=_uniform24(seed, _T_UNI_D, Rq),
                    verify_uniforms=_uniform24(seed, _T_UNI_V, Rp), notes=notes)


def position_major(w: Workload):
    """Re-lays the draft rows as [K_max, B, V] with sequences sorted by decreasing K_i, the layout a
    serving loop produces (one [B, V] logits buffer per draft step; finished sequences drop out of
    the tail of the batch).  Returns (order, q_pm, active) where order[k] is the original sequence
    in slot k and active[j] is the number of sequences still drafting at step j."""
    order = np.argsort(-w.draft_len.astype(np.int64), kind="stable")
    K = int(w.draft_len.max())
    q_pm = np.zeros((K, w.B, w.V), dtype=w.q_logits.dtype)
    for k, i in enumerate(order):
        Ki = int(w.draft_len[i])
        r0 = int(w.cu_rows[i]) - int(i)
        q_pm[:Ki, k] = w.q_logits[r0:r0 + Ki]
    active = np.array([(w.draft_len > j).sum() for j in range(K)], dtype=np.int64)
    return order, q_pm, active
