"""ctypes binding of libpeagle.so: argument marshalling only.

Every function here has the name and argument order of its C entry point in ``include/peagle.h``
and forwards device pointers of torch tensors (torch is used for device memory and streams,
nothing else).  There is no fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpeagle.so")

PEAGLE_OK = 0
STATUS = {
    "OK": 0, "NULL": -1, "BAD_SHAPE": -2, "BAD_RANGE": -3, "BAD_META": -4, "UNSUPPORTED_ARCH": -5,
    "WORKSPACE": -6, "TIMEOUT": -7, "TOO_LARGE": -8, "CUDA": -9, "ALIGN": -10,
}

EXPORTS = [
    "peagle_create", "peagle_destroy", "peagle_status_string", "peagle_last_cuda_error",
    "peagle_tile_shape", "peagle_poll_status", "peagle_launch_count", "peagle_attn_fwd",
    "peagle_attn_bwd", "peagle_attn_partitioned", "peagle_attn_partitioned_host",
    "peagle_assign_segments", "peagle_classify_tiles", "peagle_mask_dense",
    "peagle_timing_enable", "peagle_timing_read", "peagle_attn_fwd_static",
    "peagle_rope_qkv_fwd", "peagle_rope_qkv_bwd", "peagle_attn_partitioned_acc", "peagle_cast_grads",
    "peagle_gemm_bf16", "peagle_layer_partitioned", "peagle_selftest_wait_expiry",
]


class peagle_range_t(ctypes.Structure):
    _fields_ = [("begin", ctypes.c_int32), ("end", ctypes.c_int32)]


class peagle_problem_t(ctypes.Structure):
    _fields_ = [
        ("num_seqs", ctypes.c_int32),
        ("cu_seqlens", ctypes.POINTER(ctypes.c_int32)),
        ("total_tokens", ctypes.c_int32),
        ("anchor", ctypes.c_void_p),
        ("depth", ctypes.c_void_p),
        ("K", ctypes.c_int32),
        ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
    ]


class peagle_partition_t(ctypes.Structure):
    _fields_ = [
        ("seq", ctypes.c_int32),
        ("q", peagle_range_t),
        ("k", ctypes.POINTER(peagle_range_t)),
        ("nk", ctypes.c_int32),
    ]


_lib = None


def lib():
    """Loads libpeagle.so; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with __graft_entry__.build() "
                               "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        L.peagle_status_string.restype = ctypes.c_char_p
        L.peagle_last_cuda_error.restype = ctypes.c_char_p
        L.peagle_last_cuda_error.argtypes = [ctypes.c_void_p]
        L.peagle_launch_count.restype = ctypes.c_int64
        L.peagle_launch_count.argtypes = [ctypes.c_void_p]
        _lib = L
    return _lib


class PeagleError(RuntimeError):
    def __init__(self, status: int, ctx=None):
        self.status = status
        msg = lib().peagle_status_string(status).decode()
        if ctx is not None and status == STATUS["CUDA"]:
            msg += ": " + lib().peagle_last_cuda_error(ctx).decode()
        super().__init__(f"peagle status {status}: {msg}")


def _check(rc: int, ctx=None):
    if rc != PEAGLE_OK:
        raise PeagleError(rc, ctx)


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array / None."""
    if t is None:
        return ctypes.c_void_p(0)
    if isinstance(t, np.ndarray):
        return ctypes.c_void_p(t.ctypes.data)
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if hasattr(stream, "cuda_stream"):
        return ctypes.c_void_p(stream.cuda_stream)
    return ctypes.c_void_p(int(stream))


class Problem:
    """Owns the host arrays a peagle_problem_t points to."""

    def __init__(self, cu_seqlens, anchor, depth, K, n_q_heads, n_kv_heads, head_dim,
                 softmax_scale):
        self.cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
        self.anchor, self.depth = anchor, depth          # device tensors (host arrays for *_host)
        self.c = peagle_problem_t(
            len(self.cu) - 1, self.cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
            int(self.cu[-1]) if len(self.cu) else 0, _ptr(anchor), _ptr(depth), int(K),
            int(n_q_heads), int(n_kv_heads), int(head_dim), float(softmax_scale))

    def ref(self):
        return ctypes.byref(self.c)


class Partition:
    """Owns the host range array a peagle_partition_t points to."""

    def __init__(self, seq, q, k=None):
        k = [] if k is None else list(k)
        self.kr = (peagle_range_t * max(len(k), 1))(*[peagle_range_t(int(b), int(e)) for b, e in k])
        self.c = peagle_partition_t(int(seq), peagle_range_t(int(q[0]), int(q[1])),
                                    ctypes.cast(self.kr, ctypes.POINTER(peagle_range_t)) if k else None,
                                    len(k))

    def ref(self):
        return ctypes.byref(self.c)


def _partition_array(parts):
    arr = (peagle_partition_t * max(len(parts), 1))()
    for i, p in enumerate(parts):
        arr[i] = p.c
    return arr


class Context:
    def __init__(self, device: int = 0):
        self.h = ctypes.c_void_p()
        _check(lib().peagle_create(ctypes.byref(self.h), int(device)))

    def close(self):
        if self.h:
            lib().peagle_destroy(self.h)
            self.h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def peagle_tile_shape(ctx: Context, head_dim: int):
    bm, bn = ctypes.c_int(), ctypes.c_int()
    _check(lib().peagle_tile_shape(ctx.h, int(head_dim), ctypes.byref(bm), ctypes.byref(bn)))
    return bm.value, bn.value


def peagle_poll_status(ctx: Context, stream=None) -> int:
    return int(lib().peagle_poll_status(ctx.h, _stream(stream)))


def peagle_launch_count(ctx: Context) -> int:
    return int(lib().peagle_launch_count(ctx.h))


def peagle_timing_enable(ctx: Context, on: bool):
    _check(lib().peagle_timing_enable(ctx.h, int(bool(on))))


def peagle_timing_read(ctx: Context):
    """((forward ms, backward ms), (forward launches, backward launches)) since the last read."""
    ms = (ctypes.c_double * 2)()
    n = (ctypes.c_int64 * 2)()
    _check(lib().peagle_timing_read(ctx.h, ms, n), ctx.h)
    return (ms[0], ms[1]), (n[0], n[1])


def peagle_attn_fwd(ctx, prob: Problem, part: Partition, Q, K, V, O, LSE, stream=None):
    _check(lib().peagle_attn_fwd(ctx.h, prob.ref(), part.ref(), _ptr(Q), _ptr(K), _ptr(V), _ptr(O),
                                 _ptr(LSE), _stream(stream)), ctx.h)


def peagle_attn_fwd_static(device: int, prob: Problem, part: Partition, Q, K, V, O, LSE,
                           dev_status=None, stream=None):
    """Forward without any device allocation: the call's tile plan lives in a fixed array inside
    the library (4 MiB per GPU), so no context is needed.  ``dev_status`` is an optional int32
    device tensor that receives a device-side error code."""
    _check(lib().peagle_attn_fwd_static(int(device), prob.ref(), part.ref(), _ptr(Q), _ptr(K),
                                        _ptr(V), _ptr(O), _ptr(LSE), _ptr(dev_status),
                                        _stream(stream)))


def peagle_attn_bwd(ctx, prob: Problem, part: Partition, Q, K, V, O, dO, LSE, dQ, dK_acc, dV_acc,
                    stream=None):
    _check(lib().peagle_attn_bwd(ctx.h, prob.ref(), part.ref(), _ptr(Q), _ptr(K), _ptr(V), _ptr(O),
                                 _ptr(dO), _ptr(LSE), _ptr(dQ), _ptr(dK_acc), _ptr(dV_acc),
                                 _stream(stream)), ctx.h)


def peagle_attn_partitioned(ctx, prob: Problem, parts, Q, K, V, dO, O, LSE, dQ, dK, dV, stream=None):
    arr = _partition_array(parts)
    _check(lib().peagle_attn_partitioned(ctx.h, prob.ref(), arr, len(parts), _ptr(Q), _ptr(K),
                                         _ptr(V), _ptr(dO), _ptr(O), _ptr(LSE), _ptr(dQ), _ptr(dK),
                                         _ptr(dV), _stream(stream)), ctx.h)


def peagle_attn_partitioned_acc(ctx, prob: Problem, parts, Q, K, V, dO, O, LSE, dQ, dK_acc, dV_acc,
                                stream=None):
    """Forward + backward of ``parts`` adding into the caller's fp32 dK / dV accumulators."""
    arr = _partition_array(parts)
    _check(lib().peagle_attn_partitioned_acc(ctx.h, prob.ref(), arr, len(parts), _ptr(Q), _ptr(K),
                                             _ptr(V), _ptr(dO), _ptr(O), _ptr(LSE), _ptr(dQ),
                                             _ptr(dK_acc), _ptr(dV_acc), _stream(stream)), ctx.h)


def peagle_cast_grads(ctx, dK_acc, dV_acc, dK, dV, stream=None):
    """Rounds fp32 dK / dV sums to bf16."""
    _check(lib().peagle_cast_grads(ctx.h, _ptr(dK_acc), _ptr(dV_acc), ctypes.c_int64(dK_acc.numel()),
                                   _ptr(dK), _ptr(dV), _stream(stream)), ctx.h)


def peagle_attn_partitioned_host(ctx, prob: Problem, parts, Q, K, V, dO, O, LSE, dQ, dK, dV):
    """All tensors (and prob.anchor / prob.depth) are HOST memory here."""
    arr = _partition_array(parts)
    _check(lib().peagle_attn_partitioned_host(ctx.h, prob.ref(), arr, len(parts), _ptr(Q), _ptr(K),
                                              _ptr(V), _ptr(dO), _ptr(O), _ptr(LSE), _ptr(dQ),
                                              _ptr(dK), _ptr(dV)), ctx.h)


def peagle_rope_qkv_fwd(ctx, qkv, anchor, depth, Hq, Hkv, D, rope_base, Q, K, V, stream=None):
    """Rotary prologue: fused rows [T, (Hq + 2 Hkv) * D] -> Q, K (rotated), V (copied); device tensors."""
    _check(lib().peagle_rope_qkv_fwd(ctx.h, _ptr(qkv), _ptr(anchor), _ptr(depth),
                                     int(qkv.shape[0]), int(Hq), int(Hkv), int(D),
                                     ctypes.c_float(rope_base), _ptr(Q), _ptr(K), _ptr(V),
                                     _stream(stream)), ctx.h)


def peagle_rope_qkv_bwd(ctx, dQ, dK, dV, anchor, depth, Hq, Hkv, D, rope_base, d_qkv, stream=None):
    """Backward of the rotary prologue: dQ, dK, dV -> gradient of the fused rows; device tensors."""
    _check(lib().peagle_rope_qkv_bwd(ctx.h, _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(anchor), _ptr(depth),
                                     int(dQ.shape[0]), int(Hq), int(Hkv), int(D),
                                     ctypes.c_float(rope_base), _ptr(d_qkv), _stream(stream)), ctx.h)


def peagle_gemm_bf16(ctx, A, lda, a_t, B, ldb, b_t, C, ldc, c_f32_add, M, N, K, stream=None):
    """C[m][n] (+)= sum_k A(m,k) B(n,k); see include/peagle.h for the layouts."""
    _check(lib().peagle_gemm_bf16(ctx.h, _ptr(A), ctypes.c_int64(lda), int(a_t), _ptr(B),
                                  ctypes.c_int64(ldb), int(b_t), _ptr(C), ctypes.c_int64(ldc),
                                  int(c_f32_add), int(M), int(N), int(K), _stream(stream)), ctx.h)


def peagle_layer_partitioned(ctx, prob: Problem, parts, X, W, rope_base, dO, O, LSE, dX, dW, stream=None):
    """Projection -> rotary -> attention forward and backward, one pass per segment (device tensors)."""
    arr = _partition_array(parts)
    _check(lib().peagle_layer_partitioned(ctx.h, prob.ref(), arr, len(parts), _ptr(X), _ptr(W),
                                          int(X.shape[1]), ctypes.c_float(rope_base), _ptr(dO), _ptr(O),
                                          _ptr(LSE), _ptr(dX), _ptr(dW), _stream(stream)), ctx.h)


def peagle_selftest_wait_expiry(ctx, limit_ms: int = 20, stream=None):
    """Runs one bounded wait into its time limit; poll_status then reports TIMEOUT once."""
    _check(lib().peagle_selftest_wait_expiry(ctx.h, int(limit_ms), _stream(stream)), ctx.h)


def peagle_assign_segments(anchor, depth, K, boundaries):
    """Algorithm 1 on the host (no GPU needed): segment index of every token of one sequence."""
    anchor = np.ascontiguousarray(np.asarray(anchor, dtype=np.int32))
    depth = np.ascontiguousarray(np.asarray(depth, dtype=np.int32))
    b = np.ascontiguousarray(np.asarray(boundaries, dtype=np.int32))
    out = np.zeros(anchor.shape[0], np.int32)
    i32p = ctypes.POINTER(ctypes.c_int32)
    _check(lib().peagle_assign_segments(anchor.ctypes.data_as(i32p), depth.ctypes.data_as(i32p),
                                        int(anchor.shape[0]), int(K), b.ctypes.data_as(i32p),
                                        int(b.shape[0] - 1), out.ctypes.data_as(i32p)))
    return out


def peagle_classify_tiles(ctx, prob: Problem, part: Partition):
    nq, nk = ctypes.c_int32(), ctypes.c_int32()
    _check(lib().peagle_classify_tiles(ctx.h, prob.ref(), part.ref(), None, ctypes.byref(nq),
                                       ctypes.byref(nk)), ctx.h)
    out = np.zeros((nq.value, nk.value), np.uint8)
    _check(lib().peagle_classify_tiles(ctx.h, prob.ref(), part.ref(), _ptr(out), ctypes.byref(nq),
                                       ctypes.byref(nk)), ctx.h)
    return out


def peagle_mask_dense(ctx, prob: Problem, part: Partition):
    q_len = part.c.q.end - part.c.q.begin
    out = np.zeros((q_len, prob.c.total_tokens), np.uint8)
    _check(lib().peagle_mask_dense(ctx.h, prob.ref(), part.ref(), _ptr(out)), ctx.h)
    return out
