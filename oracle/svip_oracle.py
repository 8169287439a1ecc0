"""ctypes front end of the plain-C fp64 oracle (``svip_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline timing of the benchmark.  The product (the CUDA library and its
binding) never imports this module.

Logit arrays are numpy: ``float32`` for fp32 logits, ``uint16`` for bfloat16
bit patterns.  All arithmetic happens in the C file; this module only
marshals arguments, loops over rows / sequences (optionally on several host
threads -- ctypes releases the GIL) and builds the shared object with gcc.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "svip_oracle.c")
_LIB = os.path.join(_HERE, "libsvip_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile svip_oracle.c with gcc (strict IEEE fp64: no -ffast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        dp = C.POINTER(C.c_double)
        L.svip_oracle_argmax.restype = C.c_long
        L.svip_oracle_argmax.argtypes = [C.c_void_p, C.c_int, C.c_long]
        L.svip_oracle_softmax.restype = None
        L.svip_oracle_softmax.argtypes = [C.c_void_p, C.c_int, C.c_long, C.c_double, dp]
        L.svip_oracle_entropy.restype = C.c_double
        L.svip_oracle_entropy.argtypes = [dp, C.c_long]
        L.svip_oracle_invcdf.restype = C.c_long
        L.svip_oracle_invcdf.argtypes = [dp, C.c_long, C.c_double]
        L.svip_oracle_draft_step.restype = C.c_int
        L.svip_oracle_draft_step.argtypes = [
            C.c_void_p, C.c_int, C.c_long, C.c_double, C.c_double, C.c_double,
            C.POINTER(C.c_long), dp, C.POINTER(C.c_int)]
        L.svip_oracle_verify.restype = C.c_int
        L.svip_oracle_verify.argtypes = [
            C.c_long, C.c_void_p, C.c_void_p, C.c_long, C.c_void_p, C.c_long,
            C.c_int, C.c_long, C.c_double, dp,
            C.POINTER(C.c_long), C.POINTER(C.c_long), dp]
        for name in ("svip_oracle_beta", "svip_oracle_tvd", "svip_oracle_cross_entropy"):
            f = getattr(L, name)
            f.restype = C.c_double
            f.argtypes = [dp, dp, C.c_long]
        L.svip_oracle_pair_stats.restype = C.c_int
        L.svip_oracle_pair_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_long, C.c_double, C.c_double, dp]
        L.svip_oracle_threshold.restype = C.c_int
        L.svip_oracle_threshold.argtypes = [C.c_void_p, C.c_int, C.c_long, C.c_double, C.c_long, C.c_double,
                                            dp, dp, dp, C.POINTER(C.c_long)]
        L.svip_oracle_verify_tree.restype = C.c_int
        L.svip_oracle_verify_tree.argtypes = [
            C.c_long, C.c_void_p, C.c_void_p, C.c_void_p, C.c_long, C.c_void_p, C.c_long,
            C.c_int, C.c_long, C.c_double, dp, C.POINTER(C.c_long), C.c_void_p, C.POINTER(C.c_long), dp, dp]
        L.svip_oracle_residual.restype = C.c_double
        L.svip_oracle_residual.argtypes = [dp, dp, C.c_long, dp]
        _lib = L
    return _lib


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError("logits must be float32 or uint16 (bfloat16 bits), got %s" % a.dtype)


def _dptr(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _rows2d(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.ndim == 1:
        a = a[None, :]
    assert a.ndim == 2
    return a


def softmax(row: np.ndarray, T: float = 1.0) -> np.ndarray:
    row = np.ascontiguousarray(row)
    out = np.empty(row.shape[-1], dtype=np.float64)
    lib().svip_oracle_softmax(row.ctypes.data, _dtype_code(row), row.shape[-1], float(T), _dptr(out))
    return out


def entropy(prob: np.ndarray) -> float:
    prob = np.ascontiguousarray(prob, dtype=np.float64)
    return float(lib().svip_oracle_entropy(_dptr(prob), prob.size))


def invcdf(w: np.ndarray, u: float) -> int:
    w = np.ascontiguousarray(w, dtype=np.float64)
    return int(lib().svip_oracle_invcdf(_dptr(w), w.size, float(u)))


def argmax(row: np.ndarray) -> int:
    row = np.ascontiguousarray(row)
    return int(lib().svip_oracle_argmax(row.ctypes.data, _dtype_code(row), row.shape[-1]))


def beta(p, q) -> float:
    p = np.ascontiguousarray(p, dtype=np.float64); q = np.ascontiguousarray(q, dtype=np.float64)
    return float(lib().svip_oracle_beta(_dptr(p), _dptr(q), p.size))


def tvd(p, q) -> float:
    p = np.ascontiguousarray(p, dtype=np.float64); q = np.ascontiguousarray(q, dtype=np.float64)
    return float(lib().svip_oracle_tvd(_dptr(p), _dptr(q), p.size))


def cross_entropy(q, p) -> float:
    p = np.ascontiguousarray(p, dtype=np.float64); q = np.ascontiguousarray(q, dtype=np.float64)
    return float(lib().svip_oracle_cross_entropy(_dptr(q), _dptr(p), p.size))


def residual(p, q):
    p = np.ascontiguousarray(p, dtype=np.float64); q = np.ascontiguousarray(q, dtype=np.float64)
    w = np.empty_like(p)
    S = float(lib().svip_oracle_residual(_dptr(p), _dptr(q), p.size, _dptr(w)))
    return w, S


def _pmap(fn, n, threads):
    if threads <= 1 or n <= 1:
        for i in range(n):
            fn(i)
        return
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(fn, range(n)))


def draft_step(logits: np.ndarray, T: float, h: float, uniforms: np.ndarray, threads: int = 1):
    """Rows of ``logits`` [B,V] -> (token int64[B], entropy float64[B], stop uint8[B])."""
    logits = _rows2d(logits)
    B, V = logits.shape
    code = _dtype_code(logits)
    u = np.ascontiguousarray(uniforms, dtype=np.float64).reshape(B)
    token = np.empty(B, dtype=np.int64)
    H = np.empty(B, dtype=np.float64)
    stop = np.empty(B, dtype=np.uint8)
    L = lib()
    base = logits.ctypes.data
    rowbytes = logits.strides[0]

    def one(b):
        tok = C.c_long(); ent = C.c_double(); st = C.c_int()
        rc = L.svip_oracle_draft_step(base + b * rowbytes, code, V, float(T), float(h), float(u[b]),
                                      C.byref(tok), C.byref(ent), C.byref(st))
        if rc != 0:
            raise MemoryError("oracle draft_step")
        token[b] = tok.value; H[b] = ent.value; stop[b] = st.value

    _pmap(one, B, threads)
    return token, H, stop


def verify(draft_tokens: np.ndarray, q_logits: np.ndarray, target_logits: np.ndarray,
           cu_rows: np.ndarray, T: float, uniforms: np.ndarray,
           q_row_of=None, want_accept_prob: bool = False, threads: int = 1):
    """One verification round for a batch.

    ``cu_rows`` int[B+1] is the exclusive prefix of (K_i+1): target row of
    (i,j) is ``cu_rows[i]+j``; ``uniforms`` is indexed like target rows.
    Draft-side arrays (``draft_tokens``, rows of ``q_logits``) are indexed by
    ``q_row_of(i, j)``; the default is the packed layout ``cu_rows[i]-i+j``.
    Returns (n_accepted int64[B], next_token int64[B], accept_prob list | None).
    """
    q_logits = _rows2d(q_logits)
    target_logits = _rows2d(target_logits)
    V = target_logits.shape[1]
    code = _dtype_code(target_logits)
    assert _dtype_code(q_logits) == code and q_logits.shape[1] == V
    cu = np.asarray(cu_rows, dtype=np.int64)
    B = cu.size - 1
    toks = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    u = np.ascontiguousarray(uniforms, dtype=np.float64)
    n_acc = np.empty(B, dtype=np.int64)
    nxt = np.empty(B, dtype=np.int64)
    aprob = [None] * B
    L = lib()
    esz = target_logits.itemsize

    def one(i):
        K = int(cu[i + 1] - cu[i] - 1)
        if q_row_of is None:
            rows = np.arange(K, dtype=np.int64) + (cu[i] - i)
        else:
            rows = np.array([q_row_of(i, j) for j in range(K)], dtype=np.int64)
        # the C routine wants one stride between consecutive draft rows
        qstride_rows = int(rows[1] - rows[0]) if K > 1 else 1
        assert K == 1 or np.all(np.diff(rows) == qstride_rows)
        xi = np.ascontiguousarray(toks[rows])
        ri = np.ascontiguousarray(u[cu[i]:cu[i] + K + 1])
        a = np.empty(K, dtype=np.float64) if want_accept_prob else None
        na = C.c_long(); nx = C.c_long()
        rc = L.svip_oracle_verify(
            K, xi.ctypes.data,
            q_logits.ctypes.data + int(rows[0]) * q_logits.strides[0], qstride_rows * V,
            target_logits.ctypes.data + int(cu[i]) * target_logits.strides[0], V,
            code, V, float(T), _dptr(ri), C.byref(na), C.byref(nx),
            _dptr(a) if a is not None else None)
        if rc != 0:
            raise MemoryError("oracle verify")
        assert esz in (2, 4)
        n_acc[i] = na.value; nxt[i] = nx.value; aprob[i] = a

    _pmap(one, B, threads)
    return n_acc, nxt, (aprob if want_accept_prob else None)


def verify_tree(parent: np.ndarray, tokens: np.ndarray, q_logits: np.ndarray, target_logits: np.ndarray,
                T: float, uniforms: np.ndarray, want_accept_prob: bool = False, threads: int = 1,
                final_weights: np.ndarray | None = None):
    """Tree (multi-candidate) verification of B sequences with N candidate nodes each.

    ``parent`` and ``tokens`` are int [B,N] (parent -1 = child of the root, else a lower node index);
    ``q_logits`` and ``target_logits`` are [B*(N+1),V]: row b*(N+1) belongs to the root of sequence b, row
    b*(N+1)+1+i to its node i.  ``uniforms`` is [B,N+1]: an accept draw per node, then the final draw.
    Returns (n_accepted int64[B], path int32[B,N] padded with -1, next_token int64[B], accept_prob | None).
    ``final_weights``, a float64 [B,V] array, receives the unnormalised weights each next token was drawn from.
    """
    parent = np.ascontiguousarray(parent, dtype=np.int32); tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    B, N = parent.shape
    q_logits = _rows2d(q_logits); target_logits = _rows2d(target_logits)
    V = target_logits.shape[1]
    code = _dtype_code(target_logits)
    assert _dtype_code(q_logits) == code and q_logits.shape == target_logits.shape == (B * (N + 1), V)
    u = np.ascontiguousarray(uniforms, dtype=np.float64).reshape(B, N + 1)
    n_acc = np.zeros(B, dtype=np.int64); nxt = np.zeros(B, dtype=np.int64)
    path = np.full((B, max(N, 1)), -1, dtype=np.int32)
    aprob = np.full((B, max(N, 1)), -1.0) if want_accept_prob else None
    L = lib()

    def one(b):
        na = C.c_long(); nx = C.c_long()
        rc = L.svip_oracle_verify_tree(
            N, parent[b].ctypes.data, tokens[b].ctypes.data,
            q_logits.ctypes.data + b * (N + 1) * q_logits.strides[0], V,
            target_logits.ctypes.data + b * (N + 1) * target_logits.strides[0], V,
            code, V, float(T), _dptr(u[b]), C.byref(na), path[b].ctypes.data, C.byref(nx),
            C.cast(aprob[b].ctypes.data, C.POINTER(C.c_double)) if aprob is not None else None,
            C.cast(final_weights[b].ctypes.data, C.POINTER(C.c_double)) if final_weights is not None else None)
        if rc != 0:
            raise MemoryError("oracle verify_tree")
        n_acc[b] = na.value; nxt[b] = nx.value

    _pmap(one, B, threads)
    return n_acc, path[:, :N], nxt, aprob[:, :N] if aprob is not None else None


def pair_stats(target_logits: np.ndarray, q_logits: np.ndarray, T: float, c_bound: float, threads: int = 1):
    """Rows of the two [n,V] arrays pairwise -> float64 [n,8]:
    beta, H_q, H_qp, KL(q||p), gamma, Pinsker bound, Bretagnolle-Huber bound, approximation bound."""
    t = _rows2d(target_logits); q = _rows2d(q_logits)
    n, V = t.shape
    code = _dtype_code(t)
    assert q.shape == t.shape and _dtype_code(q) == code
    out = np.empty((n, 8), dtype=np.float64)
    L = lib()

    def one(r):
        rc = L.svip_oracle_pair_stats(t.ctypes.data + r * t.strides[0], q.ctypes.data + r * q.strides[0], code, V,
                                      float(T), float(c_bound),
                                      C.cast(out.ctypes.data + r * out.strides[0], C.POINTER(C.c_double)))
        if rc != 0:
            raise MemoryError("oracle pair_stats")

    _pmap(one, n, threads)
    return out


def pack_ragged(draft_len):
    """Exclusive prefix of (K_i+1) and the row -> (sequence, position) maps, by plain loops."""
    cu = [0]
    row_seq, row_pos = [], []
    for i, K in enumerate(draft_len):
        for j in range(int(K) + 1):
            row_seq.append(i)
            row_pos.append(j)
        cu.append(cu[-1] + int(K) + 1)
    return (np.array(cu, dtype=np.int64), np.array(row_seq, dtype=np.int64),
            np.array(row_pos, dtype=np.int64))


# ---------------------------------------------------------------- top-k / nucleus truncation

def threshold(logits: np.ndarray, T: float, top_k: int, top_p: float, threads: int = 1):
    """Per row: (tau, Z_topk, Z_kept, n_kept) of the truncation (see svip_oracle_threshold): the kept set is
    {i : l_i >= tau}; masses are relative to the row maximum."""
    logits = _rows2d(logits)
    n, V = logits.shape
    code = _dtype_code(logits)
    tau = np.empty(n); Zk = np.empty(n); Zt = np.empty(n); kept = np.empty(n, dtype=np.int64)
    L = lib()

    def one(r):
        a = C.c_double(); b = C.c_double(); c = C.c_double(); k = C.c_long()
        rc = L.svip_oracle_threshold(logits.ctypes.data + r * logits.strides[0], code, V, float(T), int(top_k),
                                     float(top_p), C.byref(a), C.byref(b), C.byref(c), C.byref(k))
        if rc != 0:
            raise MemoryError("oracle threshold")
        tau[r] = a.value; Zk[r] = b.value; Zt[r] = c.value; kept[r] = k.value

    _pmap(one, n, threads)
    return tau, Zk, Zt, kept


def mask_below(logits: np.ndarray, tau: np.ndarray) -> np.ndarray:
    """Copy of the rows with every logit below its row's tau replaced by -inf (dropped tokens)."""
    logits = _rows2d(logits)
    tau = np.asarray(tau, dtype=np.float64).reshape(-1, 1)
    if logits.dtype == np.float32:
        return np.where(logits.astype(np.float64) >= tau, logits, np.float32(-np.inf)).astype(np.float32)
    vals = (logits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return np.where(vals >= tau, logits, np.uint16(0xFF80)).astype(np.uint16)


def truncate(logits: np.ndarray, T: float, top_k: int, top_p: float, threads: int = 1) -> np.ndarray:
    tau, _, _, _ = threshold(logits, T, top_k, top_p, threads)
    return mask_below(logits, tau)


def draft_step_filtered(logits, T, h, uniforms, top_k, top_p, threads: int = 1):
    """The draft step on the truncated distribution: token ~ q~, H = H(q~), stop = sqrt(H) > h."""
    return draft_step(truncate(logits, T, top_k, top_p, threads), T, h, uniforms, threads)


def verify_filtered(draft_tokens, q_logits, target_logits, cu_rows, T, uniforms, top_k, top_p, q_row_of=None,
                    want_accept_prob=False, threads: int = 1):
    """The verification round with both models' distributions truncated the same way."""
    return verify(draft_tokens, truncate(q_logits, T, top_k, top_p, threads),
                  truncate(target_logits, T, top_k, top_p, threads), cu_rows, T, uniforms, q_row_of=q_row_of,
                  want_accept_prob=want_accept_prob, threads=threads)
