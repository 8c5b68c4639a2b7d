"""Shared helpers of the GPU parity tests: put a seeded case on the device, call the library
through its C ABI, and compare with the fp64 CPU oracle."""
import numpy as np
import torch

from oracle import peagle_oracle as orc
from paper_2602_01469_b200 import binding, inputs

# Tolerances of the parity contract (bf16 inputs, fp32 accumulation, bf16 outputs).
TOL_MAXABS_O = 1e-2
TOL_RELL2_O = 5e-3
TOL_RELL2_GRAD = 1e-2


def rel_l2(got, want):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    den = np.linalg.norm(want.ravel())
    return float(np.linalg.norm((got - want).ravel()) / den) if den > 0 else float(
        np.linalg.norm(got.ravel()))


class DeviceCase:
    """A laid-out workload with its tensors on cuda:0 and output buffers poisoned with NaN."""

    def __init__(self, w: inputs.Workload, q_std=None, anchor=None, depth=None, cu=None, parts=None):
        self.w = w
        if anchor is None:
            cu, anchor, depth, parts = inputs.build_case(w, binding.peagle_assign_segments)
        self.cu, self.anchor, self.depth, self.parts = cu, anchor, depth, parts
        T = int(cu[-1])
        self.T = T
        self.Q, self.K, self.V, self.dO = inputs.make_tensors(T, w.n_q_heads, w.n_kv_heads,
                                                              w.head_dim, w.seed, q_std=q_std)
        dev = torch.device("cuda:0")
        self.dQ_, self.dK_, self.dV_, self.ddO = (t.to(dev) for t in (self.Q, self.K, self.V, self.dO))
        self.d_anchor = torch.from_numpy(anchor).to(dev)
        self.d_depth = torch.from_numpy(depth).to(dev)
        nan = float("nan")
        self.O = torch.full((T, w.n_q_heads, w.head_dim), nan, dtype=torch.bfloat16, device=dev)
        self.LSE = torch.full((w.n_q_heads, T), nan, dtype=torch.float32, device=dev)
        self.dQ = torch.full_like(self.O, nan)
        self.dK = torch.full((T, w.n_kv_heads, w.head_dim), nan, dtype=torch.bfloat16, device=dev)
        self.dV = torch.full_like(self.dK, nan)
        self.prob = binding.Problem(cu, self.d_anchor, self.d_depth, w.K, w.n_q_heads, w.n_kv_heads,
                                    w.head_dim, w.scale)
        self.bparts = [binding.Partition(p["seq"], p["q"], p["k"]) for p in parts]

    def seq_slice(self, s):
        return slice(int(self.cu[s]), int(self.cu[s + 1]))

    def oracle_fwd(self, part, rows=None, heads=None):
        """Oracle O, LSE for rows (global indices) of one partition."""
        sl = self.seq_slice(part["seq"])
        off = sl.start
        rows = np.arange(*part["q"]) if rows is None else np.asarray(rows)
        kr = [(b - off, e - off) for b, e in part["k"]]
        return orc.attn_fwd(self.anchor[sl], self.depth[sl], self.Q[sl], self.K[sl], self.V[sl],
                            self.w.scale, rows=rows - off, kranges=kr, heads=heads)

    def oracle_bwd(self, part, rows=None, heads=None, dK=None, dV=None):
        sl = self.seq_slice(part["seq"])
        off = sl.start
        rows = np.arange(*part["q"]) if rows is None else np.asarray(rows)
        kr = [(b - off, e - off) for b, e in part["k"]]
        return orc.attn_bwd(self.anchor[sl], self.depth[sl], self.Q[sl], self.K[sl], self.V[sl],
                            self.dO[sl], self.w.scale, rows=rows - off, kranges=kr, heads=heads,
                            dK=dK, dV=dV)


def check_forward(got_O, got_LSE, want_O, want_LSE):
    """got_O [rows][H][D], got_LSE [rows][H] against the oracle's."""
    got_O = np.asarray(got_O, np.float64)
    got_LSE = np.asarray(got_LSE, np.float64)
    assert np.isfinite(got_O).all(), "O has NaN/inf"
    finite = np.isfinite(want_LSE)
    assert np.array_equal(np.isneginf(got_LSE), np.isneginf(want_LSE))
    assert np.abs(got_O - want_O).max() <= TOL_MAXABS_O
    assert np.abs(got_LSE[finite] - want_LSE[finite]).max() <= TOL_MAXABS_O
    assert rel_l2(got_O, want_O) <= TOL_RELL2_O
    assert rel_l2(got_LSE[finite], want_LSE[finite]) <= TOL_RELL2_O


def check_rows(name, got, want, tol=TOL_RELL2_GRAD):
    """Per-row bound beside the whole-tensor norm: every row (first axis) has relative L2 error
    <= tol, or -- for rows whose true value is close to zero -- a largest error <= tol times the
    largest magnitude of the whole tensor.  A handful of wrong rows among thousands passes a
    whole-tensor norm; it does not pass this."""
    got = np.asarray(got, np.float64).reshape(got.shape[0], -1)
    want = np.asarray(want, np.float64).reshape(want.shape[0], -1)
    assert np.isfinite(got).all(), name
    err = np.linalg.norm(got - want, axis=1)
    ref = np.linalg.norm(want, axis=1)
    floor = tol * np.abs(want).max()
    bad = (err > tol * ref) & (np.abs(got - want).max(axis=1) > floor)
    assert not bad.any(), (name, int(bad.sum()), np.nonzero(bad)[0][:8].tolist(),
                           float((err / np.maximum(ref, 1e-300))[bad].max()))
