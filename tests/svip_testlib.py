"""Shared helpers of the GPU parity tests: device marshalling, oracle-side guard bands and the
boundary predicates of the stated tolerances.

Tolerances (the numbers every parity test uses):
  ENTROPY_ATOL    entropy agrees within 1e-4 nats (fp32 accumulation against the fp64 oracle)
  CDF_TOL         a sampled token may differ from the oracle's only if the uniform lies within 1e-5
                  (in units of the total weight) of that token's own interval of the oracle's fp64
                  CDF, i.e. only across a CDF boundary closer than 1e-5; such cases are counted
                  and reported (flat tails of a 256000-token row have boundaries every ~1e-7)
  ACCEPT_GUARD    accept draws closer than 1e-4 to the oracle's acceptance probability are moved
                  away before both sides see them, so accept counts must then be bit-exact
  STOP_GUARD      stop flags must be bit-exact wherever |sqrt(H) - h| > 1e-3 (oracle value)
"""
from __future__ import annotations

import numpy as np

ENTROPY_ATOL = 1e-4
CDF_TOL = 1e-5
ACCEPT_GUARD = 1e-4
STOP_GUARD = 1e-3


def torch_mod():
    import torch
    return torch


def to_device(a: np.ndarray):
    """numpy -> CUDA tensor with the same bytes (uint16 bf16 bits travel as int16)."""
    torch = torch_mod()
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(a).cuda()


def dtype_code(a: np.ndarray) -> int:
    return 1 if a.dtype == np.uint16 else 0


def gpu_draft_step(ctx, logits: np.ndarray, T, h, uniforms, want_stats=True, pad_elems=0, row_stride=None):
    """Runs svip_draft_step on `logits` [B,V].  pad_elems shifts the first row by that many
    elements and row_stride (elements) spreads the rows, to exercise unaligned rows."""
    torch = torch_mod()
    B, V = logits.shape
    stride = V if row_stride is None else row_stride
    buf = np.zeros(pad_elems + B * stride + 16, dtype=logits.dtype)
    if logits.dtype == np.float32:
        buf[:] = np.nan       # poison the gaps: anything read outside a row shows up
    else:
        buf[:] = 0x7FC0
    for b in range(B):
        buf[pad_elems + b * stride: pad_elems + b * stride + V] = logits[b]
    dbuf = to_device(buf)
    esz = logits.itemsize
    u = to_device(np.asarray(uniforms, dtype=np.float32)) if uniforms is not None else None
    token = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    ent = torch.full((B,), -1.0, dtype=torch.float32, device="cuda")
    stop = torch.full((B,), 9, dtype=torch.uint8, device="cuda")
    stats = torch.zeros((B, 2), dtype=torch.float32, device="cuda") if want_stats else None
    ctx.draft_step(dbuf.data_ptr() + pad_elems * esz, dtype_code(logits), B, V, stride, T, h, u, token, ent,
                   stop, stats, None)
    torch.cuda.synchronize()
    return (token.cpu().numpy(), ent.cpu().numpy(), stop.cpu().numpy(),
            stats.cpu().numpy() if want_stats else None)


def gpu_verify(ctx, draft_tokens, q_logits, target_logits, cu_rows, K, T, uniforms, q_stats=None,
               fixed_K=False, layout="packed", q_seq_stride=None, q_pos_stride=None, early_exit=False):
    """svip_verify; with early_exit also svip_verify_early_exit on the same buffers: returns (plain, early)."""
    torch = torch_mod()
    B = len(cu_rows) - 1
    Rp, V = target_logits.shape
    d_tok = to_device(np.asarray(draft_tokens, dtype=np.int32))
    d_q = to_device(q_logits) if q_logits is not None else None
    d_t = to_device(target_logits)
    d_cu = None if fixed_K else to_device(np.asarray(cu_rows, dtype=np.int32))
    d_u = to_device(np.asarray(uniforms, dtype=np.float32)) if uniforms is not None else None
    d_qs = to_device(np.asarray(q_stats, dtype=np.float32)) if q_stats is not None else None
    n_acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    if layout == "packed":
        qs, qp = -1, 0
    else:
        qs, qp = q_seq_stride, q_pos_stride
    ctx.verify(d_tok, d_q, V, d_qs, qs, qp, d_t, V, dtype_code(target_logits), d_cu, B, K, Rp, V, T, d_u,
               n_acc, nxt, None)
    torch.cuda.synchronize()
    got = n_acc.cpu().numpy(), nxt.cpu().numpy()
    if not early_exit:
        return got
    # the early-exit entry point on the same buffers
    n_acc.fill_(-7); nxt.fill_(-7)
    ctx.verify_early_exit(d_tok, d_q, V, d_qs, qs, qp, d_t, V, dtype_code(target_logits), d_cu, B, K, Rp, V, T, d_u,
                          n_acc, nxt, None)
    torch.cuda.synchronize()
    return got, (n_acc.cpu().numpy(), nxt.cpu().numpy())


# ---------------------------------------------------------------- oracle-side guard bands / predicates

def guard_accept_uniforms(oracle, draft_tokens, q_logits, target_logits, cu_rows, T, uniforms, threads=8):
    """Moves every accept draw that lies within ACCEPT_GUARD of the oracle's acceptance probability
    to the far side of the guard band (deterministic).  Returns (uniforms, number moved)."""
    u = np.array(uniforms, dtype=np.float32, copy=True)
    if not T > 0:
        return u, 0
    _, _, aprob = oracle.verify(draft_tokens, q_logits, target_logits, cu_rows, T, u.astype(np.float64),
                                want_accept_prob=True, threads=threads)
    moved = 0
    for i, a in enumerate(aprob):
        r0 = int(cu_rows[i])
        for j, aj in enumerate(a):
            if aj >= 1.0:
                continue            # r < 1 always accepts; no boundary inside [0,1)
            r = float(u[r0 + j])
            if abs(r - aj) < ACCEPT_GUARD:
                new = aj + 2 * ACCEPT_GUARD if r >= aj else aj - 2 * ACCEPT_GUARD
                if new >= 1.0:
                    new = aj - 2 * ACCEPT_GUARD
                if new < 0.0:
                    new = aj + 2 * ACCEPT_GUARD
                u[r0 + j] = np.float32(new)
                moved += 1
    return u, moved


def within_cdf_tolerance(weights: np.ndarray, u: float, token: int, tol: float = CDF_TOL) -> bool:
    """True if `token` is what the inverse CDF returns for some u' with |u' - u| <= tol, i.e. if
    u * total lies within tol * total of the token's own interval [c_{token-1}, c_token) of the fp64
    cumulative sums, and the token has positive weight."""
    c = np.cumsum(weights.astype(np.float64))
    total = c[-1]
    if not total > 0 or not (0 <= token < len(c)) or not weights[token] > 0:
        return False
    lo = (c[token - 1] if token > 0 else 0.0) / total
    hi = c[token] / total
    return bool(lo - tol <= float(u) <= hi + tol)


def check_draft_against_oracle(oracle, logits, T, h, uniforms, got, label="", threads=8):
    """Compares (token, entropy, stop) with the oracle row by row; returns counters."""
    tok_g, H_g, stop_g, _ = got
    tok_o, H_o, stop_o = oracle.draft_step(logits, T, h, uniforms if uniforms is not None else
                                           np.zeros(logits.shape[0]), threads=threads)
    err = np.abs(H_g.astype(np.float64) - H_o)
    assert np.all(err <= ENTROPY_ATOL), "%s entropy off by %g at row %d" % (label, err.max(), err.argmax())
    off_boundary = np.abs(np.sqrt(H_o) - h) > STOP_GUARD
    assert np.array_equal(stop_g[off_boundary], stop_o[off_boundary]), label + " stop flags differ"
    counters = {"rows": len(tok_o), "stop_near_threshold": int((~off_boundary).sum()), "token_boundary": 0}
    bad = np.nonzero(tok_g.astype(np.int64) != tok_o)[0]
    if not T > 0:
        assert bad.size == 0, "%s greedy tokens differ at rows %s" % (label, bad[:8])
        return counters
    for b in bad:
        q = oracle.softmax(logits[b], T)
        assert within_cdf_tolerance(q, uniforms[b], int(tok_g[b])), \
            "%s row %d: token %d vs oracle %d, beyond the CDF tolerance" % (label, b, tok_g[b], tok_o[b])
        counters["token_boundary"] += 1
    return counters


def check_verify_against_oracle(oracle, draft_tokens, q_logits, target_logits, cu_rows, T, uniforms, got,
                                label="", q_row_of=None, threads=8):
    n_g, nx_g = got
    n_o, nx_o, _ = oracle.verify(draft_tokens, q_logits, target_logits, cu_rows, T,
                                 np.asarray(uniforms if uniforms is not None else
                                            np.zeros(int(cu_rows[-1])), dtype=np.float64),
                                 q_row_of=q_row_of, threads=threads)
    assert np.array_equal(n_g.astype(np.int64), n_o), "%s n_accepted differs: %s vs %s" % (
        label, n_g[:16], n_o[:16])
    counters = {"sequences": len(n_o), "next_boundary": 0, "mean_accepted": float(n_o.mean())}
    bad = np.nonzero(nx_g.astype(np.int64) != nx_o)[0]
    if not T > 0:
        assert bad.size == 0, label + " greedy next tokens differ"
        return counters
    for i in bad:
        r0 = int(cu_rows[i]); K = int(cu_rows[i + 1]) - r0 - 1
        p = oracle.softmax(target_logits[r0 + n_o[i]], T)
        if n_o[i] < K:
            dr = (r0 - i + n_o[i]) if q_row_of is None else q_row_of(int(i), int(n_o[i]))
            w, S = oracle.residual(p, oracle.softmax(q_logits[dr], T))
            if not S > 0:
                w = p
        else:
            w = p
        assert within_cdf_tolerance(w, uniforms[r0 + K], int(nx_g[i])), \
            "%s seq %d: next %d vs oracle %d, beyond the CDF tolerance" % (label, i, nx_g[i], nx_o[i])
        counters["next_boundary"] += 1
    return counters
