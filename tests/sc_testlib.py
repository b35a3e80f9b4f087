"""Glue for the parity tests: runs one workload through the CUDA library (via the C ABI binding) and
through the CPU oracle on the same seeded inputs.  The two sides meet only here."""
import numpy as np

from paper_2609_32922_b200 import workloads as wl

MODES = {"bipolar": 0, "unipolar": 1}
SCALES = {"none": 0, "per_row": 1, "per_tensor": 2}

REL_TOL = 1e-6      # decoded fp32 outputs: relative tolerance ...
ABS_TOL = 1e-7      # ... with this absolute floor (popcounts are compared bit-exactly)


def close_enough(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return np.all(np.abs(got - ref) <= np.maximum(REL_TOL * np.abs(ref), ABS_TOL))


def gpu_params(binding, w, group=1, core=0):
    return binding.make_params(mode=MODES[w.mode], scale_a=SCALES[w.scale_a], scale_w=SCALES[w.scale_w],
                               group=group, seed=w.seed, stream_id=w.stream_id, core=core)


def gpu_matmul(sc, binding, w, A, W, L_groups, Lmax, group=1, core=0, want_P=True):
    """L_groups: numpy int32 per group, or None for uniform Lmax.  Returns numpy (P, C)."""
    import torch
    dA = torch.from_numpy(A).cuda()
    dW = torch.from_numpy(W).cuda()
    dL = None if L_groups is None else torch.from_numpy(np.ascontiguousarray(L_groups, dtype=np.int32)).cuda()
    P, C = sc.matmul(dA, dW, dL, Lmax, gpu_params(binding, w, group, core), want_P=want_P)
    torch.cuda.synchronize()
    return (None if P is None else P.cpu().numpy()), C.cpu().numpy()


def oracle_matmul(oracle, w, A, W, L_rows, rows=None, cols=None, quant=0):
    return oracle.matmul(A, W, L_rows, MODES[w.mode], SCALES[w.scale_a], SCALES[w.scale_w], w.seed, w.stream_id,
                         row_sel=rows, col_sel=cols, quant=quant)


def policy_lengths(oracle, w, A):
    """Per-group lengths of a policy workload, from the oracle's Sec. 4.4 assignment."""
    avg, Lmin, Lmax, group = w.policy
    g = oracle.row_absmax(A)
    L, realised = oracle.assign_lengths(g, group, avg, Lmin, Lmax)
    return L, realised
