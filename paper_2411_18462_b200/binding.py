"""ctypes binding of the C ABI in ``include/svip.h``: argument marshalling only.

Every method of :class:`Context` has the name and the argument order of the C
function it calls.  Device buffers may be given as ``torch`` CUDA tensors (their
``data_ptr()`` is passed) or as integer device addresses; ``stream`` may be a
``torch.cuda.Stream``, an integer ``cudaStream_t`` or ``None`` (the legacy
default stream).  Nothing here computes: if the compiled library is missing the
import of a symbol fails with :class:`SvipError`.
"""
from __future__ import annotations

import ctypes as C
import os

SVIP_F32 = 0
SVIP_BF16 = 1
SVIP_Q_PACKED = -1
SVIP_STATUS_NONFINITE_ROW = 1
SVIP_STATUS_BAD_DRAFT_LEN = 2
SVIP_STATUS_WAIT_TIMEOUT = 4
SVIP_STATUS_BAD_TREE = 8

_HERE = os.path.dirname(os.path.abspath(__file__))
# SVIP_LIBRARY in the environment points at another build of the same ABI (a debug build, say)
_LIB_PATH = os.environ.get("SVIP_LIBRARY") or os.path.join(_HERE, "csrc", "libsvip.so")
_lib = None


class SvipError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__("svip: %s (status %d)" % (text, code))
        self.code = code


def library_path() -> str:
    return _LIB_PATH


def library():
    """Loads csrc/libsvip.so (built by ``python -m paper_2411_18462_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise SvipError(-100, "CUDA library %s is not built; run python -m paper_2411_18462_b200.build"
                        % _LIB_PATH)
    L = C.CDLL(_LIB_PATH)
    vp, i32, lng, f32 = C.c_void_p, C.c_int, C.c_long, C.c_float
    L.svip_strerror.restype = C.c_char_p
    L.svip_strerror.argtypes = [i32]
    L.svip_version.restype = i32
    L.svip_version.argtypes = []
    L.svip_last_cuda_error.restype = i32
    L.svip_last_cuda_error.argtypes = [vp]
    L.svip_create.restype = i32
    L.svip_create.argtypes = [C.POINTER(vp), i32, i32]
    L.svip_destroy.restype = i32
    L.svip_destroy.argtypes = [vp]
    L.svip_set_cluster_size.restype = i32
    L.svip_set_cluster_size.argtypes = [vp, i32]
    L.svip_launch_count.restype = lng
    L.svip_launch_count.argtypes = [vp]
    L.svip_read_status.restype = i32
    L.svip_read_status.argtypes = [vp, C.POINTER(C.c_uint), vp]
    L.svip_draft_step.restype = i32
    L.svip_draft_step.argtypes = [vp, vp, i32, i32, i32, lng, f32, f32, vp, vp, vp, vp, vp, vp]
    L.svip_pack_ragged.restype = i32
    L.svip_pack_ragged.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    L.svip_verify.restype = i32
    L.svip_verify.argtypes = [vp, vp, vp, lng, vp, lng, lng, vp, lng, i32, vp, i32, i32, i32, i32, f32,
                              vp, vp, vp, vp]
    L.svip_verify_early_exit.restype = i32
    L.svip_verify_early_exit.argtypes = [vp, vp, vp, lng, vp, lng, lng, vp, lng, i32, vp, i32, i32, i32, i32, f32,
                              vp, vp, vp, vp]
    L.svip_profile_enable.restype = i32
    L.svip_profile_enable.argtypes = [vp, i32]
    L.svip_profile_read.restype = i32
    L.svip_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_long)]
    L.svip_pair_stats_given.restype = i32
    L.svip_pair_stats_given.argtypes = [vp, vp, lng, vp, vp, lng, vp, i32, i32, i32, f32, f32, vp, vp]
    L.svip_verify_tree.restype = i32
    L.svip_verify_tree.argtypes = [vp, vp, vp, vp, lng, vp, vp, lng, i32, i32, i32, i32, f32, vp, vp, vp, vp, vp]
    L.svip_selftest_wait_timeout.restype = i32
    L.svip_selftest_wait_timeout.argtypes = [vp, lng, vp]
    L.svip_draft_step_masked.restype = i32
    L.svip_draft_step_masked.argtypes = [vp, vp, i32, i32, i32, lng, f32, f32, vp, vp, vp, vp, vp, vp, vp]
    L.svip_draft_step_at.restype = i32
    L.svip_draft_step_at.argtypes = [vp, vp, i32, i32, i32, lng, lng, vp, lng, f32, f32, vp, vp, vp, vp, vp, vp, vp]
    L.svip_graph_loop_begin.restype = i32
    L.svip_graph_loop_begin.argtypes = [vp, vp, vp, i32, C.POINTER(vp)]
    L.svip_graph_loop_end.restype = i32
    L.svip_graph_loop_end.argtypes = [vp]
    L.svip_row_threshold.restype = i32
    L.svip_row_threshold.argtypes = [vp, vp, i32, i32, i32, lng, f32, i32, f32, vp, vp, vp]
    L.svip_draft_step_filtered.restype = i32
    L.svip_draft_step_filtered.argtypes = [vp, vp, i32, i32, i32, lng, f32, f32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.svip_draft_step_truncated.restype = i32
    L.svip_draft_step_truncated.argtypes = [vp, vp, i32, i32, i32, lng, f32, f32, i32, f32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.svip_verify_filtered.restype = i32
    L.svip_verify_filtered.argtypes = [vp, vp, vp, lng, vp, vp, lng, lng, vp, lng, vp, vp, i32, vp, i32, i32, i32,
                                       i32, f32, vp, vp, vp, vp]
    L.svip_policy_advance.restype = i32
    L.svip_policy_advance.argtypes = [vp, i32, vp, vp, vp, vp, i32, i32, vp, vp]
    L.svip_policy_update.restype = i32
    L.svip_policy_update.argtypes = [vp, i32, vp, vp, vp, vp, i32, i32, vp]
    L.svip_vp_partial.restype = i32
    L.svip_vp_partial.argtypes = [vp, vp, i32, i32, i32, lng, f32, i32, vp, vp]
    L.svip_vp_combine.restype = i32
    L.svip_vp_combine.argtypes = [vp, vp, i32, i32, i32, f32, f32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.svip_vp_locate.restype = i32
    L.svip_vp_locate.argtypes = [vp, vp, i32, i32, i32, lng, f32, vp, vp, i32, vp, vp]
    L.svip_pair_stats.restype = i32
    L.svip_pair_stats.argtypes = [vp, vp, lng, vp, lng, i32, i32, i32, f32, f32, vp, vp]
    L.svip_verify_noalloc.restype = i32
    L.svip_verify_noalloc.argtypes = [i32, vp, vp, lng, vp, lng, lng, vp, lng, i32, vp, i32, i32, i32, i32, f32,
                                      vp, vp, vp, vp, vp]
    L.svip_graph_begin.restype = i32
    L.svip_graph_begin.argtypes = [vp, vp]
    L.svip_graph_end.restype = i32
    L.svip_graph_end.argtypes = [vp, vp, C.POINTER(vp)]
    L.svip_graph_launch.restype = i32
    L.svip_graph_launch.argtypes = [vp, vp]
    L.svip_graph_destroy.restype = i32
    L.svip_graph_destroy.argtypes = [vp]
    _lib = L
    return L


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(s):
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _check(code: int, ctx=None):
    if code != 0:
        text = library().svip_strerror(code).decode()
        if code == -4 and ctx is not None:
            text += " (cudaError %d)" % library().svip_last_cuda_error(ctx)
        raise SvipError(code, text)


def verify_noalloc(device, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                   target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                   n_accepted, next_token, status=None, stream=None):
    """``svip_verify_noalloc``: the verify round without a context and without any allocation."""
    _check(library().svip_verify_noalloc(int(device), _ptr(draft_tokens), _ptr(q_logits), int(q_row_stride),
                                         _ptr(q_stats), int(q_seq_stride), int(q_pos_stride),
                                         _ptr(target_logits), int(t_row_stride), int(dtype), _ptr(cu_rows),
                                         int(B), int(K), int(n_target_rows), int(V), float(T), _ptr(uniforms),
                                         _ptr(n_accepted), _ptr(next_token), _ptr(status), _stream(stream)))


class Graph:
    def __init__(self, handle):
        self._h = handle

    def launch(self, stream=None):
        _check(library().svip_graph_launch(self._h, _stream(stream)))

    def destroy(self):
        if self._h:
            library().svip_graph_destroy(self._h)
            self._h = None


class Context:
    """Owns an ``svip_ctx``; methods mirror the C functions one to one."""

    def __init__(self, device: int = 0, max_rows: int = 1 << 15):
        self._h = C.c_void_p()
        _check(library().svip_create(C.byref(self._h), int(device), int(max_rows)))

    def destroy(self):
        if self._h:
            library().svip_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def set_cluster_size(self, cluster_size: int):
        _check(library().svip_set_cluster_size(self._h, int(cluster_size)))

    def launch_count(self) -> int:
        return int(library().svip_launch_count(self._h))

    def read_status(self, stream=None) -> int:
        flags = C.c_uint(0)
        _check(library().svip_read_status(self._h, C.byref(flags), _stream(stream)), self._h)
        return int(flags.value)

    def draft_step(self, logits, dtype, B, V, row_stride, T, thresh, uniforms, token, entropy, stop,
                   row_stats=None, stream=None):
        _check(library().svip_draft_step(self._h, _ptr(logits), int(dtype), int(B), int(V), int(row_stride),
                                         float(T), float(thresh), _ptr(uniforms), _ptr(token), _ptr(entropy),
                                         _ptr(stop), _ptr(row_stats), _stream(stream)), self._h)

    def draft_step_masked(self, logits, dtype, B, V, row_stride, T, thresh, uniforms, active, token, entropy, stop,
                          row_stats=None, stream=None):
        _check(library().svip_draft_step_masked(self._h, _ptr(logits), int(dtype), int(B), int(V), int(row_stride),
                                                float(T), float(thresh), _ptr(uniforms), _ptr(active), _ptr(token),
                                                _ptr(entropy), _ptr(stop), _ptr(row_stats), _stream(stream)),
               self._h)

    def draft_step_at(self, logits, dtype, B, V, row_stride, pos_stride, pos, slot_stride, T, thresh, uniforms,
                      active, token, entropy, stop, row_stats=None, stream=None):
        _check(library().svip_draft_step_at(self._h, _ptr(logits), int(dtype), int(B), int(V), int(row_stride),
                                            int(pos_stride), _ptr(pos), int(slot_stride), float(T), float(thresh),
                                            _ptr(uniforms), _ptr(active), _ptr(token), _ptr(entropy), _ptr(stop),
                                            _ptr(row_stats), _stream(stream)), self._h)

    def row_threshold(self, logits, dtype, n_rows, V, row_stride, T, top_k, top_p, thr, stats=None, stream=None):
        _check(library().svip_row_threshold(self._h, _ptr(logits), int(dtype), int(n_rows), int(V), int(row_stride),
                                            float(T), int(top_k), float(top_p), _ptr(thr), _ptr(stats),
                                            _stream(stream)), self._h)

    def draft_step_filtered(self, logits, dtype, B, V, row_stride, T, thresh, uniforms, active, thr, token, entropy,
                            stop, row_stats=None, stream=None):
        _check(library().svip_draft_step_filtered(self._h, _ptr(logits), int(dtype), int(B), int(V), int(row_stride),
                                                  float(T), float(thresh), _ptr(uniforms), _ptr(active), _ptr(thr),
                                                  _ptr(token), _ptr(entropy), _ptr(stop), _ptr(row_stats),
                                                  _stream(stream)), self._h)

    def draft_step_truncated(self, logits, dtype, B, V, row_stride, T, thresh, top_k, top_p, uniforms, active, thr,
                             token, entropy, stop, row_stats=None, stream=None):
        _check(library().svip_draft_step_truncated(self._h, _ptr(logits), int(dtype), int(B), int(V), int(row_stride),
                                                   float(T), float(thresh), int(top_k), float(top_p), _ptr(uniforms),
                                                   _ptr(active), _ptr(thr), _ptr(token), _ptr(entropy), _ptr(stop),
                                                   _ptr(row_stats), _stream(stream)), self._h)

    def verify_filtered(self, draft_tokens, q_logits, q_row_stride, q_stats, q_thr, q_seq_stride, q_pos_stride,
                        target_logits, t_row_stride, p_thr, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                        n_accepted, next_token, p_stats=None, stream=None):
        _check(library().svip_verify_filtered(
            self._h, _ptr(draft_tokens), _ptr(q_logits), int(q_row_stride), _ptr(q_stats), _ptr(q_thr),
            int(q_seq_stride), int(q_pos_stride), _ptr(target_logits), int(t_row_stride), _ptr(p_thr),
            _ptr(p_stats), int(dtype),
            _ptr(cu_rows), int(B), int(K), int(n_target_rows), int(V), float(T), _ptr(uniforms), _ptr(n_accepted),
            _ptr(next_token), _stream(stream)), self._h)

    def policy_advance(self, policy, stop, gamma, draft_len, active, B, K_cap, n_active=None, stream=None):
        _check(library().svip_policy_advance(self._h, int(policy), _ptr(stop), _ptr(gamma), _ptr(draft_len),
                                             _ptr(active), int(B), int(K_cap), _ptr(n_active), _stream(stream)),
               self._h)

    def policy_update(self, policy, n_accepted, draft_len, gamma, active, B, K_cap, stream=None):
        _check(library().svip_policy_update(self._h, int(policy), _ptr(n_accepted), _ptr(draft_len), _ptr(gamma),
                                            _ptr(active), int(B), int(K_cap), _stream(stream)), self._h)

    def pack_ragged(self, draft_len, B, K_max, cu_rows, row_seq=None, row_pos=None, stream=None):
        _check(library().svip_pack_ragged(self._h, _ptr(draft_len), int(B), int(K_max), _ptr(cu_rows),
                                          _ptr(row_seq), _ptr(row_pos), _stream(stream)), self._h)

    def verify(self, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
               target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
               n_accepted, next_token, stream=None):
        _check(library().svip_verify(self._h, _ptr(draft_tokens), _ptr(q_logits), int(q_row_stride),
                                     _ptr(q_stats), int(q_seq_stride), int(q_pos_stride),
                                     _ptr(target_logits), int(t_row_stride), int(dtype), _ptr(cu_rows),
                                     int(B), int(K), int(n_target_rows), int(V), float(T), _ptr(uniforms),
                                     _ptr(n_accepted), _ptr(next_token), _stream(stream)), self._h)

    def verify_early_exit(self, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                          target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                          n_accepted, next_token, stream=None):
        _check(library().svip_verify_early_exit(self._h, _ptr(draft_tokens), _ptr(q_logits), int(q_row_stride),
                                                _ptr(q_stats), int(q_seq_stride), int(q_pos_stride),
                                                _ptr(target_logits), int(t_row_stride), int(dtype), _ptr(cu_rows),
                                                int(B), int(K), int(n_target_rows), int(V), float(T),
                                                _ptr(uniforms), _ptr(n_accepted), _ptr(next_token),
                                                _stream(stream)), self._h)

    def vp_partial(self, logits, dtype, B, V_shard, row_stride, T, vocab_offset, partial, stream=None):
        _check(library().svip_vp_partial(self._h, _ptr(logits), int(dtype), int(B), int(V_shard), int(row_stride),
                                         float(T), int(vocab_offset), _ptr(partial), _stream(stream)), self._h)

    def vp_combine(self, partials, G, rank, B, T, thresh, uniforms, entropy, stop, token, owner, local_target,
                   active, stream=None):
        _check(library().svip_vp_combine(self._h, _ptr(partials), int(G), int(rank), int(B), float(T), float(thresh),
                                         _ptr(uniforms), _ptr(entropy), _ptr(stop), _ptr(token), _ptr(owner),
                                         _ptr(local_target), _ptr(active), _stream(stream)), self._h)

    def vp_locate(self, logits, dtype, B, V_shard, row_stride, T, local_target, active, vocab_offset, token,
                  stream=None):
        _check(library().svip_vp_locate(self._h, _ptr(logits), int(dtype), int(B), int(V_shard), int(row_stride),
                                        float(T), _ptr(local_target), _ptr(active), int(vocab_offset), _ptr(token),
                                        _stream(stream)), self._h)

    def pair_stats(self, q_logits, q_row_stride, target_logits, t_row_stride, dtype, n_pairs, V, T, c_bound, out,
                   stream=None):
        _check(library().svip_pair_stats(self._h, _ptr(q_logits), int(q_row_stride), _ptr(target_logits),
                                         int(t_row_stride), int(dtype), int(n_pairs), int(V), float(T),
                                         float(c_bound), _ptr(out), _stream(stream)), self._h)

    def verify_tree(self, tokens, parent, q_logits, q_row_stride, q_stats, target_logits, t_row_stride, dtype, B, N, V,
                    T, uniforms, n_accepted, path, next_token, stream=None):
        _check(library().svip_verify_tree(self._h, _ptr(tokens), _ptr(parent), _ptr(q_logits), int(q_row_stride),
                                          _ptr(q_stats), _ptr(target_logits), int(t_row_stride), int(dtype), int(B),
                                          int(N), int(V), float(T), _ptr(uniforms), _ptr(n_accepted), _ptr(path),
                                          _ptr(next_token), _stream(stream)), self._h)

    def pair_stats_given(self, q_logits, q_row_stride, q_stats, target_logits, t_row_stride, p_stats, dtype, n_pairs, V, T,
                         c_bound, out, stream=None):
        _check(library().svip_pair_stats_given(self._h, _ptr(q_logits), int(q_row_stride), _ptr(q_stats),
                                               _ptr(target_logits), int(t_row_stride), _ptr(p_stats), int(dtype),
                                               int(n_pairs), int(V), float(T), float(c_bound), _ptr(out),
                                               _stream(stream)), self._h)

    def selftest_wait_timeout(self, wait_ns: int, stream=None):
        _check(library().svip_selftest_wait_timeout(self._h, int(wait_ns), _stream(stream)), self._h)

    def profile_enable(self, on: bool):
        _check(library().svip_profile_enable(self._h, 1 if on else 0), self._h)

    def profile_read(self):
        ms = C.c_double(0.0)
        n = C.c_long(0)
        _check(library().svip_profile_read(self._h, C.byref(ms), C.byref(n)), self._h)
        return float(ms.value), int(n.value)

    def bind(self, name: str, *args):
        """Pre-marshals one call: returns a zero-argument callable that runs ``svip_<name>(ctx, *args)``
        and raises on a non-zero status.  Saves the per-call conversion cost in launch-bound loops."""
        fn = getattr(library(), "svip_" + name)
        conv = []
        for a, t in zip(args, fn.argtypes[1:]):
            if t is C.c_void_p:
                a = _ptr(a) if not hasattr(a, "cuda_stream") else a.cuda_stream
                conv.append(C.c_void_p(a))
            else:
                conv.append(t(a))
        h = self._h
        conv = tuple(conv)

        def call():
            rc = fn(h, *conv)
            if rc != 0:
                _check(rc, h)
        return call

    def graph_begin(self, stream):
        _check(library().svip_graph_begin(self._h, _stream(stream)), self._h)

    def graph_loop_begin(self, stream, n_active, max_iters) -> int:
        """Opens the loop body; returns the raw stream handle on which the body is recorded."""
        body = C.c_void_p()
        _check(library().svip_graph_loop_begin(self._h, _stream(stream), _ptr(n_active), int(max_iters),
                                               C.byref(body)), self._h)
        return int(body.value)

    def graph_loop_end(self):
        _check(library().svip_graph_loop_end(self._h), self._h)

    def graph_end(self, stream) -> Graph:
        g = C.c_void_p()
        _check(library().svip_graph_end(self._h, _stream(stream), C.byref(g)), self._h)
        return Graph(g)
