"""Randomised small shapes through every entry point of the product path against the oracle: odd sizes, depth tails,
lengths from 0 upwards, both modes, every core, groups, scale kinds, prepared weights and batches."""
import dataclasses

import numpy as np
import pytest

from paper_2609_32922_b200 import workloads as wl
import sc_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2609_32922_b200 import build, binding as b
    build.build()
    return b


@pytest.fixture(scope="module")
def sc(binding):
    s = binding.ScGemm(0)
    yield s
    assert s.device_status() == 0
    s.close()


@pytest.mark.parametrize("case", range(30))
def test_random_single_products(sc, binding, oracle, case):
    import torch
    rng = np.random.default_rng(1000 + case)
    M, K, N = int(rng.integers(1, 300)), int(rng.integers(1, 200)), int(rng.integers(1, 420))
    Lmax = int(rng.choice([1, 7, 32, 33, 64, 100]))
    mode = ["bipolar", "unipolar"][case % 2]
    core = [0, 1, 2, 3, 4, 5][case % 6] if case < 24 else 5
    group = int(rng.choice([1, 1, 3, 8]))
    w, _ = wl.small_ragged(seed=case, M=M, K=K, N=N, mode=mode, Lmax=Lmax)
    w = dataclasses.replace(w, scale_a=str(rng.choice(["none", "per_row", "per_tensor"])),
                            scale_w=str(rng.choice(["none", "per_row", "per_tensor"])), stream_id=int(rng.integers(0, 5)))
    A, W = wl.make_inputs(w)
    if w.scale_a == "none":
        A = np.clip(A, -1.2, 1.2).astype(np.float32)
    W = (W * 30).astype(np.float32)                       # some weights beyond [-1, 1] when unscaled: clamped
    Lg = rng.integers(0, Lmax + 1, size=(M + group - 1) // group).astype(np.int32)
    L_rows = oracle.expand_lengths(Lg, M, group)
    ref = T.oracle_matmul(oracle, w, A, W, L_rows)
    P, C = T.gpu_matmul(sc, binding, w, A, W, Lg, Lmax, group=group, core=core)
    assert np.array_equal(P, ref["P"]), (M, K, N, Lmax, mode, core)
    assert T.close_enough(C, ref["C"])
    if case % 3 == 0:                                     # the same through prepared weights
        params = T.gpu_params(binding, w, group, core)
        dW = torch.from_numpy(W).cuda()
        prepared = sc.prepare_weights(dW, Lmax, params)
        P2, C2 = sc.matmul_prepared(torch.from_numpy(A).cuda(), prepared, torch.from_numpy(Lg).cuda(), Lmax, params)
        torch.cuda.synchronize()
        binding.sc_weights_release(prepared[0])
        assert np.array_equal(P2.cpu().numpy(), ref["P"]) and T.close_enough(C2.cpu().numpy(), ref["C"])


@pytest.mark.parametrize("case", range(10))
def test_random_batches(sc, binding, oracle, case):
    import torch
    rng = np.random.default_rng(2000 + case)
    B, M, K, N = int(rng.integers(1, 7)), int(rng.integers(1, 200)), int(rng.integers(1, 100)), int(rng.integers(1, 260))
    Lmax = int(rng.choice([5, 32, 48]))
    mode = case % 2
    transposed = bool((case // 2) % 2)
    core = [0, 2, 4, 1, 3][case % 5]
    scale_w = int(rng.choice([0, 1, 2]))
    A = rng.standard_normal((B, M, K)).astype(np.float32)
    W = rng.standard_normal((B, N, K) if transposed else (B, K, N)).astype(np.float32)
    L = rng.integers(0, Lmax + 1, size=B * M).astype(np.int32)
    params = binding.make_params(mode=mode, scale_a=1, scale_w=scale_w, seed=case, stream_id=1, core=core)
    P, C = sc.matmul_batched(torch.from_numpy(A).cuda(), torch.from_numpy(W).cuda(), transposed, torch.from_numpy(L).cuda(),
                             Lmax, params)
    torch.cuda.synchronize()
    ref = oracle.matmul_batched(A, W, L, mode, 1, scale_w, seed=case, stream_id=1, w_transposed=transposed)
    assert np.array_equal(P.cpu().numpy(), ref["P"]), (B, M, K, N, Lmax, mode, transposed, core)
    assert T.close_enough(C.cpu().numpy(), ref["C"])


@pytest.mark.parametrize("case", range(6))
def test_random_cbsg(sc, binding, oracle, case):
    import torch
    rng = np.random.default_rng(3000 + case)
    M, K, N = int(rng.integers(1, 200)), int(rng.integers(1, 120)), int(rng.integers(1, 300))
    Lmax = int(rng.choice([1, 31, 100, 256]))
    group = int(rng.choice([1, 4]))
    A = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.standard_normal((K, N)).astype(np.float32)
    Lg = rng.integers(0, Lmax + 1, size=(M + group - 1) // group).astype(np.int32)
    params = binding.make_params(mode=0, scale_a=1, scale_w=int(rng.choice([1, 2])), group=group, seed=case, stream_id=case)
    P, C = sc.matmul_cbsg(torch.from_numpy(A).cuda(), torch.from_numpy(W).cuda(), torch.from_numpy(Lg).cuda(), Lmax, params)
    torch.cuda.synchronize()
    ref = oracle.matmul_cbsg(A, W, oracle.expand_lengths(Lg, M, group), 1, params.scale_w, seed=case, stream_id=case)
    assert np.array_equal(P.cpu().numpy(), ref["P"]), (M, K, N, Lmax, group)
    assert T.close_enough(C.cpu().numpy(), ref["C"])
